"""Benchmark of the NITI integer training step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config I] [--impl ours|reference]

One "step" = one full integer training step (forward, integer cross-entropy gradient, backward,
int8 weight update; Algorithm 1 of the paper) over one synthetic batch.  Default workload:
config 4, the ImageNet-shaped VGG-16 stack at batch 64 (the largest single-GPU configuration).
Prints ONE JSON line (rank 0).  With N > 1 every rank trains its own replica on its own batch
(weak scaling, no collective on the data path).

--impl reference times the CPU oracle (the only reference there is: the paper ships no code in
this repository) on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "int8_training_images_per_sec"
UNIT = "images/s"


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_burst": d["bf16_tflops"],
                "bf16_sustained": d["bf16_tflops_sustained"], "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_burst": 1590.0, "bf16_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples nvidia-smi clocks / throttle reasons while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                 "--format=csv,noheader,nounits", "-lms", "20"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._pump, daemon=True).start()
        except Exception:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.rows.append(line.strip())

    def stop(self):
        if self.proc:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=2)
            except Exception:
                self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            f = [x.strip() for x in r.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except ValueError:
                continue
            for name, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def cpu_baseline(config: int, budget_s: float = 20.0):
    """Times the oracle, as it stands, on a bounded sample of the workload."""
    import numpy as np
    from oracle import OracleNetState, oracle_train_step, ref
    from synth import config_net, make_net_inputs
    ref.build()
    cores = ref.n_threads()
    # probe the oracle's conv rate to size the sample
    rng = np.random.default_rng(0)
    x = rng.integers(-127, 128, size=(1, 32, 32, 64), dtype=np.int8)
    w = rng.integers(-127, 128, size=(64, 3, 3, 64), dtype=np.int8)
    t0 = time.perf_counter()
    ref.conv_fwd_acc(x, w, 1)
    rate = 32 * 32 * 64 * 64 * 9 / max(time.perf_counter() - t0, 1e-6)     # MAC/s
    sample = None
    cands = {0: [(64, 1)],
             2: [(256, 1), (64, 1), (16, 1), (4, 1)],
             3: [(256, 1), (64, 1), (16, 1), (4, 1), (1, 1)],
             4: [(64, 1), (16, 1), (4, 1), (1, 1), (1, 2), (1, 4), (1, 7)]}[config]
    for batch, scale in cands:            # the largest sample that fits the time budget
        net = config_net(config, batch=batch, scale=scale)
        if 3 * net.macs_per_pass() / rate <= budget_s or (batch, scale) == cands[-1]:
            sample = (batch, scale, net)
            break
    batch, scale, net = sample
    x, labels, weights = make_net_inputs(net)
    st = OracleNetState([w.copy() for w in weights])
    t0 = time.perf_counter()
    oracle_train_step(net, x, labels, st, allow_overflow=True)
    dt = time.perf_counter() - t0
    return {"value": batch / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": "one step of %s at batch %d, image side / %d (%.2f s)" % (net.name, batch, scale, dt),
            "seconds": dt}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from synth import config_net
    vals = []
    cb = None
    for _ in range(max(1, args.warmup > 0)):
        cpu_baseline(args.config, budget_s=5.0)
    for _ in range(args.steps):
        cb = cpu_baseline(args.config, budget_s=10.0)
        vals.append(cb["value"])
    v = sum(vals) / len(vals)
    net = config_net(args.config)
    line = {"impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * cb["seconds"],
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int64",
            "data": "synthetic", "config": {"workload": "config%d:%s" % (args.config, net.name),
                                            "global_batch": net.batch},
            "cpu_baseline": {"value": v, "unit": UNIT, "cores": cb["cores"], "kind": "oracle",
                             "sample": cb["sample"]},
            "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def gemm_point(niti, M, N, K, iters=10, dist="uniform", variant="act"):
    """Fused int8 GEMM (multiply + bit-width + shift + pseudo-stochastic round) at one shape.
    variant "act": out[M,N] = a[M,K] w[N,K]^T rounded to 7 bits (forward entry point);
    variant "grad": g[M,N] = e[K,M]^T a[K,N] rounded to 5 bits (weight-gradient entry point)."""
    import torch
    from synth import gemm_grad_operands, gemm_operands
    dev = niti.device
    if variant == "act":
        a, w = gemm_operands(M, N, K, dist)
        a, w = torch.from_numpy(a).to(dev), torch.from_numpy(w).to(dev)
        sa, sw = niti.scalar(-7), niti.scalar(-10)
        out = torch.empty((M, N), dtype=torch.int8, device=dev)
        s_out, b_out = niti.scalar(), niti.scalar()      # (allocated once: no allocator call per launch)

        def run():
            niti.linear_fwd(a, sa, w, sw, out=out, s_out=s_out, b_out=b_out)
    else:
        e, a2 = gemm_grad_operands(M, N, K, dist)
        e, a2 = torch.from_numpy(e).to(dev), torch.from_numpy(a2).to(dev)
        wdummy = torch.zeros((16,), dtype=torch.int8, device=dev)
        g = torch.empty((M, N), dtype=torch.int8, device=dev)
        b_g = niti.scalar()

        def run():
            niti.linear_bwd(a2, e, wdummy, need_e_prev=False, g=g, b_g=b_g, m_u=5)
    for _ in range(3):
        run()
    torch.cuda.synchronize()
    niti.profile_enable(True)
    e0, e1 = torch.cuda.Event(True), torch.cuda.Event(True)
    e0.record()
    for _ in range(iters):
        run()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / iters
    k_ms, k_n, k_ops = niti.profile_read()
    niti.profile_enable(False)
    pk = _peaks()
    tops = 2.0 * M * N * K / ms / 1e9
    return {"shape": [M, N, K], "dist": dist, "variant": variant, "fused_ms": ms, "fused_tops": tops,
            "frac_of_2x_bf16_burst": tops / (2.0 * pk["bf16_burst"]), "frac_of_nominal_4500": tops / 4500.0,
            "mma_kernel_ms": k_ms / max(k_n, 1), "mma_kernel_tops": k_ops / max(k_ms, 1e-9) / 1e9}


def run_sweep(args):
    """Config 1: the 64-shape fused-GEMM sweep, two operand distributions, two rounding targets."""
    from paper_2009_13108_b200 import Niti
    from synth import GEMM_SWEEP_DIMS
    niti = Niti(0)
    dims = GEMM_SWEEP_DIMS
    for dist in ("uniform", "gauss"):
        for variant in ("act", "grad"):
            for M in dims:
                for N in dims:
                    for K in dims:
                        if dist == "gauss" and min(M, N, K) < 4096 and not args.full_sweep:
                            continue          # the second operand set is timed on the large shapes
                        r = gemm_point(niti, M, N, K, iters=5, dist=dist, variant=variant)
                        print(json.dumps(r), flush=True)
    print(json.dumps({"redo_passes": niti.redo_count()}), flush=True)
    niti.check()


def run_paper_table(args):
    """The layer of the paper's convolution timing table (batch 64, 64 -> 128 channels, 3x3, stride 1,
    pad 1, square inputs 224 ... 14): forward, dgrad and wgrad including bit-width, shift and rounding."""
    import numpy as np
    import torch
    from paper_2009_13108_b200 import Niti
    niti = Niti(0)
    dev = niti.device
    rng = np.random.Generator(np.random.PCG64(11))
    paper_3090_ms = {224: (3.928, 4.731, 122.301), 112: (1.006, 1.269, 27.327), 56: (0.289, 0.453, 6.911),
                     28: (0.089, 0.185, 1.074), 14: (0.038, 0.117, 0.272)}
    for side in (224, 112, 56, 28, 14):
        B, Ci, Co = 64, 64, 128
        x = torch.from_numpy(rng.integers(-127, 128, size=(B, side, side, Ci), dtype=np.int8)).to(dev)
        w = torch.from_numpy(rng.integers(-127, 128, size=(Co, 3, 3, Ci), dtype=np.int8)).to(dev)
        e = torch.from_numpy(rng.integers(-127, 128, size=(B, side, side, Co), dtype=np.int8)).to(dev)
        y, ep, g = torch.empty_like(e), torch.empty_like(x), torch.empty_like(w)
        sx, sw = niti.scalar(-7), niti.scalar(-10)
        ops = 2.0 * B * side * side * Ci * Co * 9
        row = {"input": side, "batch": B, "cin": Ci, "cout": Co, "int8_ops": ops,
               "paper_rtx3090_ms": dict(zip(("a", "e", "g"), paper_3090_ms[side]))}
        for name, fn in (("a", lambda: niti.conv_fwd(x, sx, w, sw, y=y)),
                         ("e", lambda: niti.conv_dgrad(e, w, (side, side), e_prev=ep)),
                         ("g", lambda: niti.conv_wgrad(x, e, g=g))):
            for _ in range(3):
                fn()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(True), torch.cuda.Event(True)
            e0.record()
            for _ in range(args.iters):
                fn()
            e1.record()
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1) / args.iters
            row[name + "_ms"] = ms
            row[name + "_tops"] = ops / ms / 1e9
        print(json.dumps(row), flush=True)
    niti.check()


def run_conv_shape(args):
    """One 3x3 / pad 1 convolution layer at BxHxWxCinxCout: forward (with ReLU), error (with the ReLU gate)
    and weight gradient, each timed with CUDA events; a small case for profiler captures."""
    import numpy as np
    import torch
    from paper_2009_13108_b200 import Niti
    niti = Niti(0)
    dev = niti.device
    B, H, W, Ci, Co = (int(v) for v in args.conv_shape.lower().split("x"))
    rng = np.random.Generator(np.random.PCG64(12))
    x = torch.from_numpy(np.maximum(rng.integers(-127, 128, size=(B, H, W, Ci), dtype=np.int8), 0)).to(dev)
    w = torch.from_numpy(rng.integers(-127, 128, size=(Co, 3, 3, Ci), dtype=np.int8)).to(dev)
    e = torch.from_numpy(rng.integers(-127, 128, size=(B, H, W, Co), dtype=np.int8)).to(dev)
    y, ep, g = torch.empty_like(e), torch.empty_like(x), torch.empty_like(w)
    sx, sw, sy = niti.scalar(-7), niti.scalar(-10), niti.scalar()
    b_y, b_e, b_g = niti.scalar(), niti.scalar(), niti.scalar()
    ops = 2.0 * B * H * W * Ci * Co * 9
    row = {"conv": [B, H, W, Ci, Co], "int8_ops": ops}
    for name, fn, nbytes in (
            ("fwd", lambda: niti.conv_fwd(x, sx, w, sw, y=y, s_y=sy, b_y=b_y, relu=True), x.numel() + w.numel() + y.numel()),
            ("dgrad", lambda: niti.conv_dgrad(e, w, (H, W), e_prev=ep, relu_mask_src=x, b_e=b_e),
             e.numel() + w.numel() + 2 * x.numel()),
            ("wgrad", lambda: niti.conv_wgrad(x, e, g=g, b_g=b_g), x.numel() + e.numel() + w.numel())):
        if args.only and name != args.only:
            continue
        for _ in range(2):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(True), torch.cuda.Event(True)
        e0.record()
        for _ in range(args.iters):
            fn()
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / args.iters
        row[name] = {"ms": ms, "tops": ops / ms / 1e9, "algorithmic_bytes": nbytes}
    print(json.dumps(row), flush=True)
    niti.check()


def run_elementwise(args):
    """HBM-bound kernels at sizes well beyond the 126 MB L2: achieved GB/s = algorithmic bytes / time."""
    import numpy as np
    import torch
    from paper_2009_13108_b200 import Niti
    niti = Niti(0)
    dev = niti.device
    pk = _peaks()
    gen = torch.Generator(device=dev)
    gen.manual_seed(5)

    def rnd(shape, lo=-127, hi=128):
        return torch.randint(lo, hi, shape, dtype=torch.int8, device=dev, generator=gen)

    def timeit(fn, iters=args.iters):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(True), torch.cuda.Event(True)
        e0.record()
        for _ in range(iters):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / iters

    n = 1 << 29                                   # 512 Mi elements
    w, g = rnd((n,)), rnd((n,), -31, 32)
    x = rnd((n,))
    y = torch.empty_like(x)
    B, H, W, C = 64, 224, 224, 64                  # the first pooled activation of the VGG-16 stack
    px = rnd((B, H, W, C), 0, 128)
    py = torch.empty((B, H // 2, W // 2, C), dtype=torch.int8, device=dev)
    pe = rnd((B, H // 2, W // 2, C))
    pex = torch.empty_like(px)
    logits = rnd((65536, 1000))
    labels = torch.randint(0, 1000, (65536,), dtype=torch.int32, device=dev, generator=gen)
    le = torch.empty_like(logits)
    s_a = niti.scalar(-4)
    cases = [
        ("niti_int_sgd_update", lambda: niti.int_sgd_update(w, g), 3.0 * n),
        ("niti_relu_fwd", lambda: niti.relu_fwd(x, y), 2.0 * n),
        ("niti_relu_bwd", lambda: niti.relu_bwd(x, g, y), 3.0 * n),
        ("niti_maxpool2_fwd", lambda: niti.maxpool2_fwd(px, py), 1.25 * px.numel()),
        ("niti_maxpool2_bwd", lambda: niti.maxpool2_bwd(px, pe, pex, relu=True), 2.25 * px.numel()),
        ("niti_int_xent", lambda: niti.int_xent(logits, s_a, labels, e=le), 2.0 * logits.numel() + 4.0 * 65536),
    ]
    for name, fn, nbytes in cases:
        ms = timeit(fn)
        gbs = nbytes / ms / 1e6
        print(json.dumps({"kernel": name, "algorithmic_bytes": nbytes, "ms": ms, "GB/s": gbs,
                          "frac_of_measured_hbm": gbs / pk["hbm_gbs"], "hbm_peak_GB/s": pk["hbm_gbs"],
                          "peak_source": pk["source"]}), flush=True)
    niti.check()


def run_per_launch(args):
    """One eager training step of the chosen config with a CUDA event pair around every tensor-core
    multiply (the library's own profiling hooks): one text line per multiply, in launch order."""
    import torch
    from paper_2009_13108_b200 import Niti, NitiTrainer
    from synth import config_net, make_net_inputs
    niti = Niti(0)
    net = config_net(args.config)
    x, labels, weights = make_net_inputs(net)
    tr = NitiTrainer(niti, net, weights)
    tr.load_batch(x, labels)
    tr.snapshot_weights()
    for _ in range(2):
        tr.reset_weights()
        tr.step()
    torch.cuda.synchronize()
    redo0 = niti.redo_count()
    niti.profile_enable(True)
    e0, e1 = torch.cuda.Event(True), torch.cuda.Event(True)
    tr.reset_weights()
    e0.record()
    tr.step()
    e1.record()
    torch.cuda.synchronize()
    launches = niti.profile_read_launches()
    wl = [(i, l) for i, l in enumerate(net.layers) if l["op"] != "pool"]
    names = ["fwd   L%d %s" % (i, l["op"]) for i, l in wl]
    for i, l in reversed(wl):
        # (the fused-update calls compute the error of the layer below first: it needs the old weights)
        pair = ["wgrad L%d %s" % (i, l["op"])]
        if i != wl[0][0]:
            pair.append("dgrad L%d %s" % (i, l["op"]))
        names += reversed(pair) if tr.fused_update else pair
    print("eager step %.3f ms, second passes in the step: %d" % (e0.elapsed_time(e1), niti.redo_count() - redo0))
    total = 0.0
    for k, (ms, ops) in enumerate(launches):
        total += ms
        name = names[k] if len(names) == len(launches) else ""
        print("%3d %-18s %8.1f us %7.0f TOP/s %8.1f Gop" % (k, name, ms * 1e3, ops / ms / 1e9, ops / 1e9))
    print("tensor-core multiplies: %.3f ms in %d launches" % (total, len(launches)))
    niti.check()


def algorithmic_bytes_per_multiply(net):
    """Bytes every matrix multiply of one training step must move (both operands once, the int8 result
    once, and for an error multiply the ReLU gate bytes it reads); one entry per multiply, in the order
    forward layers, then weight gradient / error of every layer from the last to the first."""
    fwd, bwd = [], []
    first = True
    shape = (net.batch,) + tuple(net.in_shape)
    for L in net.layers:
        if L["op"] == "conv":
            n_in = shape[0] * shape[1] * shape[2] * L["cin"]
            n_out = shape[0] * shape[1] * shape[2] * L["cout"]
            n_w = 9 * L["cin"] * L["cout"]
            shape = shape[:3] + (L["cout"],)
        elif L["op"] == "pool":
            shape = (shape[0], shape[1] // 2, shape[2] // 2, shape[3])
            continue
        else:
            n_in, n_out, n_w = net.batch * L["k"], net.batch * L["n"], L["k"] * L["n"]
            shape = (net.batch, L["n"])
        fwd.append(n_in + n_w + n_out)
        layer_bwd = [n_in + n_out + n_w]                 # weight gradient: activations, errors -> g
        if not first:
            layer_bwd.append(n_out + n_w + 2 * n_in)     # error: e, w -> e_prev, gated by the input's sign
        bwd.append(layer_bwd)
        first = False
    out = list(fwd)
    for lb in reversed(bwd):
        out += lb
    return out


def measured_traffic(kernel_file):
    """DRAM traffic of the dominant kernel relative to its algorithmic bytes, from the committed ncu
    summary (profiles/tc_gemm_dram_traffic.json).  The figure belongs to one build of the kernel: it is
    used only while the device code of the kernel still has the recorded SHA-256."""
    path = os.path.join(ROOT, "profiles", "tc_gemm_dram_traffic.json")
    if not os.path.exists(path):
        return None, "no committed ncu capture"
    rec = json.load(open(path))
    if rec.get("kernel_device_code_sha256") != kernel_device_digest(kernel_file):
        return None, "kernel source changed since the committed ncu capture (%s)" % rec.get("captured", "?")
    return rec, None


def kernel_device_digest(kernel_file):
    """SHA-256 of the device part of the kernel's source file: everything above its 'Host side' banner
    (the kernel, its helpers and its parameter block), so that host-only edits keep a capture valid."""
    import hashlib
    text = open(kernel_file, "rb").read()
    cut = text.find(b"// Host side: tensor maps")
    return hashlib.sha256(text if cut < 0 else text[:cut]).hexdigest()


def spawn_ranks(args):
    """`python bench.py --gpus N` without a launcher: start the N ranks here (one process per GPU,
    rendezvous on 127.0.0.1) and pass their output through."""
    from paper_2009_13108_b200.dist_util import launch_ranks
    argv = [a for a in sys.argv[1:]]
    return launch_ranks([os.path.abspath(__file__)] + argv, args.gpus)


def run_ours(args):
    import torch
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    torch.cuda.set_device(local)
    import hashlib
    import numpy as np
    from paper_2009_13108_b200 import Niti, NitiTrainer
    from paper_2009_13108_b200.build import CSRC
    from paper_2009_13108_b200 import build as _lib_build
    from synth import config_net, make_net_inputs, make_step_batch

    niti = Niti(local)
    net = config_net(args.config)
    from paper_2009_13108_b200.dist_util import aggregate_throughput, max_over_ranks, rank_seed
    net.seed = rank_seed(net.seed, rank)         # every rank draws its own batch and replica
    x, labels, weights = make_net_inputs(net)
    wh = hashlib.sha256()
    for w in weights:
        wh.update(memoryview(w).cast("B"))
    input_digests = {"x": hashlib.sha256(memoryview(x).cast("B")).hexdigest()[:16],
                     "labels": hashlib.sha256(memoryview(labels).cast("B")).hexdigest()[:16],
                     "weights": wh.hexdigest()[:16]}      # guards against drift of the seeded generator
    tr = NitiTrainer(niti, net, weights, fused_update=args.fused_update, pool_codes=args.pool_codes,
                     pool_fused=args.pool_fused)
    # Config 2 is "trained for 100 integer steps": consecutive steps on fresh mini-batches with the weights
    # carried over.  The other configs time ONE step K times: every iteration restores the seeded weights
    # (device-to-device copies inside the timed region) and repeats the same step; repeated steps on
    # random labels saturate the big nets' weights and leave the domain of the integer loss.
    train = args.config == 2
    n_batches = min(args.steps + args.warmup + 1, 128) if train else 1
    host_batches = []
    for t in range(n_batches):
        bx, bl = (x, labels) if t == 0 else make_step_batch(net, t)
        host_batches.append((torch.from_numpy(bx).pin_memory(), torch.from_numpy(bl).pin_memory()))
    dev_batches = [(bx.to(niti.device), bl.to(niti.device)) for bx, bl in host_batches]
    xh, lh = host_batches[0]
    tr.load_batch(xh, lh)
    tr.snapshot_weights()
    torch.cuda.synchronize()
    step_no = [0]

    def step_body():
        tr.step()

    def one_step():
        if train:
            bx, bl = dev_batches[step_no[0] % n_batches]       # batch already resident in HBM
            tr.load_batch(bx, bl)
            step_no[0] += 1
        else:
            tr.reset_weights()
        step_body()

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local)
    sampler.start()                               # runs through warm-up, the timed region and the e2e loop
    for _ in range(args.warmup):
        one_step()
    niti.check()
    launches_per_step = None
    if args.graph:
        # replay the captured launch sequence (same kernels, same order) instead of re-issuing it
        # from Python: removes the host-side launch cost, which dominates the small configs
        launches_per_step = niti.launch_count()
        replay = tr.capture(with_reset=not train)
        launches_per_step = niti.launch_count() - launches_per_step
        step_body = replay
        if not train:
            def one_step():                       # noqa: F811  (the graph holds the weight restore too)
                replay()
        one_step()
        niti.check()
    niti.profile_enable(not args.graph)
    # ---- device-resident timing ----
    barrier()
    l0 = niti.launch_count()
    redo0 = niti.redo_count()
    marks = [torch.cuda.Event(True) for _ in range(args.steps + 1)]
    marks[0].record()
    for i in range(args.steps):
        one_step()
        marks[i + 1].record()
    barrier()
    ms = marks[0].elapsed_time(marks[-1])
    per_step = sorted(marks[i].elapsed_time(marks[i + 1]) for i in range(args.steps))
    launches = niti.launch_count() - l0
    if args.graph:
        launches = launches_per_step * args.steps
    redo = niti.redo_count() - redo0
    niti.check()
    # digests of what the timed region left behind (the oracle-written digests of the tests are the
    # same quantities): every weight tensor and the logits
    w_sha = [hashlib.sha256(w.cpu().numpy().tobytes()).hexdigest() for w in tr.weights]
    out_digests = {"weights_sha256_16": [h[:16] for h in w_sha],
                   "weights_combined_sha256_16": hashlib.sha256("".join(w_sha).encode()).hexdigest()[:16],
                   "logits_sha256_16": hashlib.sha256(tr.acts[-1].cpu().numpy().tobytes()).hexdigest()[:16],
                   "hits_last_step": int(tr.n_correct)}
    if args.graph:
        # per-kernel timing for the roofline, in the launch configuration of the timed region: a second
        # graph of the same step, captured with the library's profiling events on (they become
        # event-record nodes around every tensor-core multiply), replayed K times; the event pairs are
        # read after every replay
        niti.profile_enable(True)
        prof_replay = tr.capture(with_reset=not train)
        k_ms, k_n, k_ops = 0.0, 0, 0.0
        for _ in range(args.steps):
            prof_replay()
            torch.cuda.synchronize()
            for t_ms, t_ops in niti.profile_read_launches():
                k_ms += t_ms
                k_ops += t_ops
                k_n += 1
        if train:
            tr.reset_weights()
        niti.profile_read()
    else:
        k_ms, k_n, k_ops = niti.profile_read()
    niti.profile_enable(False)
    # ---- end to end: host batch in, hit count out, every step ----
    result = torch.zeros(args.steps, dtype=torch.int32).pin_memory()
    read_back = [torch.cuda.Event() for _ in range(args.steps)]
    barrier()
    t0 = torch.cuda.Event(True)
    t1 = torch.cuda.Event(True)
    t0.record()
    # every step's batch comes from pinned host memory inside the timed region; the copy of the next
    # batch runs on a copy stream while the current step computes (double buffering through the
    # trainer's prefetch_batch / commit_batch); the hit count of every step is copied to the host and
    # the host waits for it one step behind, so that the next step is already queued
    tr.prefetch_batch(*host_batches[0])
    for i in range(args.steps):
        tr.commit_batch()
        if i + 1 < args.steps:
            tr.prefetch_batch(*host_batches[(i + 1) % n_batches])
        if not train and not args.graph:
            tr.reset_weights()
        step_body()
        result[i:i + 1].copy_(tr.n_correct, non_blocking=True)
        read_back[i].record()
        if i > 0:
            read_back[i - 1].synchronize()
    read_back[args.steps - 1].synchronize()
    t1.record()
    barrier()
    ms_e2e = t0.elapsed_time(t1)
    clocks = sampler.stop()
    niti.check()
    # ---- sustained: the same step replayed for seconds, so that the power cap and the clocks it
    # settles at are part of the number ----
    sustained = None
    if args.sustain_seconds > 0 and not train:
        n_sus = max(args.steps, int(args.sustain_seconds * 1e3 / (ms / args.steps)) + 1)
        s2 = ClockSampler(local)
        barrier()
        s2.start()
        e0, e1 = torch.cuda.Event(True), torch.cuda.Event(True)
        e0.record()
        for _ in range(n_sus):
            one_step()
        e1.record()
        barrier()
        sus_ms = e0.elapsed_time(e1)
        sc = s2.stop()
        niti.check()
        sustained = {"steps": n_sus, "seconds": sus_ms / 1e3, "ms_per_step": sus_ms / n_sus,
                     "value": net.batch * n_sus * world / (sus_ms / 1e3), "unit": UNIT, "clocks": sc}
    ms, ms_e2e = max_over_ranks([ms, ms_e2e], device="cuda")
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return
    pk = _peaks()
    images = net.batch * args.steps * world
    ops_step = net.int8_ops_per_step()
    # Dense int8 tensor peak = 2 x the bf16 rate measured on this machine (int8 : bf16 = 2 : 1 nominal).  The
    # dominant kernel is timed launch by launch with CUDA events in a region far shorter than a second
    # (no power capping: the clocks line shows it), so the burst measurement is its denominator; the
    # sustained one belongs to the seconds-long leg below.
    int8_peak = 2.0 * pk["bf16_burst"]
    achieved = k_ops / max(k_ms, 1e-9) / 1e9
    alg = algorithmic_bytes_per_multiply(net)
    alg_mean = sum(alg) / len(alg)
    rec, why = measured_traffic(os.path.join(CSRC, "niti_tc_gemm.cu"))
    traffic = rec["dram_bytes_per_launch"] / rec["algorithmic_bytes_per_launch"] * alg_mean if rec else None
    if sustained is not None:
        sus_tops = ops_step / sustained["ms_per_step"] / 1e9
        mhz = sustained["clocks"].get("sm_mhz")
        sustained.update({"step_tops": sus_tops, "peak": 2.0 * pk["bf16_sustained"],
                          "frac_of_2x_bf16_sustained": sus_tops / (2.0 * pk["bf16_sustained"]),
                          "ms_x_mhz": (sustained["ms_per_step"] * mhz) if mhz else None})
    line = {
        "metric": METRIC, "value": aggregate_throughput(net.batch * args.steps, ms, world), "unit": UNIT,
        "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms / args.steps,
        "ms_per_step_median": per_step[len(per_step) // 2], "ms_per_step_best": per_step[0],
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "s8",
        "data": "synthetic",
        "config": {"workload": "config%d:%s" % (args.config, net.name), "global_batch": net.batch * world,
                   "per_gpu_batch": net.batch, "int8_ops_per_step": ops_step,
                   "l2": "working set (activations + int32 scratch) exceeds the 126 MB L2",
                   "state": ("weights carried from step to step, a fresh mini-batch every step" if train else
                             "weights restored to the seeded initial values before every step"),
                   "launch": "cuda-graph replay" if args.graph else "eager",
                   "weight_update": "fused with the weight gradient" if args.fused_update else "separate call",
                   "max_pool_forward": "in the convolution's epilogue" if tr.pool_fused else "separate pass",
                   "parallelism": "replicas" if world > 1 else "single",
                   "inputs_sha256_16": input_digests},
        "outputs": out_digests,
        "library": {"sources_sha256_16": _lib_build.source_digest()[:16],
                    "built_from_these_sources": _lib_build.built_from_current_sources()},
        "step_tops": ops_step / (ms / args.steps) / 1e9,
        "clocks": clocks,
        "e2e": {"value": images / (ms_e2e / 1e3), "unit": UNIT, "h2d_bytes_per_step": int(xh.numel() + lh.numel() * 4),
                "d2h_bytes_per_step": 4},
        "gpu_launches": int(launches),
        "speculation_redo_passes": int(redo),
        "roofline": {"bound": "tensor", "kernel": "tc_gemm_kernel (tcgen05 kind::i8)", "achieved": achieved,
                     "peak": int8_peak, "unit": "TOP/s", "frac": achieved / int8_peak,
                     "peak_source": "2 x %s bf16 burst (%.1f TFLOP/s; int8 : bf16 = 2 : 1 nominal): the kernel is timed "
                                    "per launch, the region lasts %.0f ms" % (pk["source"], pk["bf16_burst"], ms),
                     "frac_of_nominal_4500": achieved / 4500.0,
                     "frac_of_measured_issue_peak_4582": achieved / 4582.0,
                     "frac_of_2x_bf16_sustained": achieved / (2.0 * pk["bf16_sustained"]),
                     "launches": k_n,
                     # DRAM bytes per multiply: the ratio DRAM bytes / algorithmic bytes of one ncu capture
                     # of a single launch (profiles/tc_gemm_dram_traffic.json) times the mean algorithmic
                     # bytes of this step's multiplies; null when the kernel changed after the capture
                     "traffic": traffic, "traffic_note": why if rec is None else rec.get("workload"),
                     "traffic_unit": "bytes per multiply (mean over the %d multiplies of the step)" % len(alg),
                     "algorithmic_bytes": alg_mean,
                     "timing": "CUDA event pair around every launch of the kernel over %d steps%s" % (
                         args.steps, " (event-record nodes in a second graph of the same step, replayed after the "
                                     "timed region)" if args.graph else "")},
    }
    if sustained is not None:
        line["sustained"] = sustained
    if args.gemm:
        line["gemm_sweep"] = [gemm_point(niti, *s) for s in [(4096, 4096, 4096), (8192, 8192, 8192)]]
    line["cpu_baseline"] = {k: v for k, v in cpu_baseline(args.config).items() if k != "seconds"}
    if args.config in (0, 2):
        line["cpu_baseline"]["single_thread"] = cpu_baseline_single_thread(args.config)
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def cpu_baseline_single_thread(config):
    """The same oracle sample on one host thread (a child process with OMP_NUM_THREADS=1)."""
    env = dict(os.environ, OMP_NUM_THREADS="1")
    for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK"):
        env.pop(k, None)
    try:
        out = subprocess.run([sys.executable, os.path.abspath(__file__), "--cpu-baseline-json", "--config", str(config)],
                             env=env, capture_output=True, text=True, timeout=180)
        d = json.loads(out.stdout.strip().splitlines()[-1])
        return {"value": d["value"], "unit": UNIT, "cores": 1, "sample": d["sample"]}
    except Exception as exc:      # the baseline is a reported extra: never fail the bench over it
        return {"unavailable": repr(exc)}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", type=int, default=4, choices=[0, 2, 3, 4])
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-gemm", dest="gemm", action="store_false")
    ap.add_argument("--no-graph", dest="graph", action="store_false",
                    help="issue every launch from Python instead of replaying a CUDA graph of the step")
    ap.add_argument("--pool-codes", dest="pool_codes", action="store_true",
                    help="max-pool forward records its routing; backward reads the codes instead of the pooled tensor")
    ap.add_argument("--separate-update", dest="fused_update", action="store_false",
                    help="weight gradient and weight update as two library calls (niti_int_sgd_update after "
                         "niti_conv_wgrad / niti_linear_bwd) instead of the fused *_update calls")
    ap.add_argument("--gemm-shape", default=None,
                    help="MxNxK: time only the fused GEMM at this shape (for profiling a small case)")
    ap.add_argument("--conv-shape", default=None,
                    help="BxHxWxCinxCout: time one 3x3 convolution layer (forward, error, weight gradient)")
    ap.add_argument("--only", default=None, choices=["fwd", "dgrad", "wgrad"], help="with --conv-shape: one of the three")
    ap.add_argument("--iters", type=int, default=10)
    ap.add_argument("--sweep", action="store_true", help="run the fused-GEMM sweep (config 1), one JSON line per point")
    ap.add_argument("--paper-table", action="store_true",
                    help="time the conv layer of the paper's timing table (fwd / dgrad / wgrad, five input sizes)")
    ap.add_argument("--elementwise", action="store_true", help="achieved GB/s of the HBM-bound kernels")
    ap.add_argument("--per-launch", action="store_true",
                    help="one eager step with a CUDA event pair around every tensor-core multiply")
    ap.add_argument("--full-sweep", action="store_true", help="with --sweep: time the second operand set on every shape")
    ap.add_argument("--no-pool-fused", dest="pool_fused", action="store_false",
                    help="separate max-pool passes in the forward step instead of pooling in the convolution's epilogue")
    ap.add_argument("--sustain-seconds", type=float, default=3.0,
                    help="also replay the step for this many seconds and report the sustained rate (0: skip)")
    ap.add_argument("--cpu-baseline-json", action="store_true", help=argparse.SUPPRESS)
    args = ap.parse_args()
    if args.cpu_baseline_json:
        print(json.dumps(cpu_baseline(args.config, budget_s=15.0)), flush=True)
        return
    if args.sweep:
        run_sweep(args)
        return
    if args.paper_table:
        run_paper_table(args)
        return
    if args.elementwise:
        run_elementwise(args)
        return
    if args.per_launch:
        run_per_launch(args)
        return
    if args.conv_shape:
        run_conv_shape(args)
        return
    if args.gemm_shape:
        from paper_2009_13108_b200 import Niti
        niti = Niti(0)
        M, N, K = (int(v) for v in args.gemm_shape.lower().split("x"))
        print(json.dumps(gemm_point(niti, M, N, K, iters=args.iters)), flush=True)
        niti.check()
        return
    if args.impl == "reference":
        run_reference(args)
    elif args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(spawn_ranks(args))
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
