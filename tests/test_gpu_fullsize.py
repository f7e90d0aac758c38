"""Parity at the benchmark's full sizes (config 4: ImageNet-shaped VGG-16, batch 64), in the
launch configuration the bench times.  The oracle cannot run these tensors whole, so it computes
sampled outputs one by one from the very operands the GPU kernel read:

* forward / dgrad: every channel of sampled output pixels, from the 3x3 input patch;
* wgrad: sampled (co, r, s, ci) entries, each a sum over all 3.2 M pixels;
* the shared bit-width b: bounded below by the sampled accumulators and pinned by the invariant
  that the shift leaves max |q| in [2^(mbits-1), 2^mbits - 1] whenever b > mbits.

Full-size config 2 and config 3 steps are compared tensor by tensor with the oracle."""
import numpy as np
import pytest
import torch

from synth import config_net, make_net_inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def niti():
    from paper_2009_13108_b200 import Niti
    n = Niti(0)
    yield n
    n.check()
    n.close()


def _psr_vec(oref, acc, bp, mbits):
    return np.array([oref.psr(int(v), bp, mbits) for v in np.asarray(acc).reshape(-1)], dtype=np.int64)


def _check_conv_fwd_samples(oref, x, w, y, b, relu, rng, n_samples=24):
    """x [B,H,W,Ci] int8 (numpy), w [Co,3,3,Ci], y GPU output (numpy), b the GPU's bit-width."""
    B, H, W, Ci = x.shape
    bp = max(0, b - 7)
    worst = 0
    # corners and edges always included
    pts = [(0, 0, 0), (B - 1, H - 1, W - 1), (B // 2, 0, W - 1), (B - 1, H - 1, 0)]
    pts += [(int(rng.integers(B)), int(rng.integers(H)), int(rng.integers(W))) for _ in range(n_samples)]
    for (bi, i, j) in pts:
        patch = np.zeros((1, 3, 3, Ci), np.int8)
        for r in range(3):
            for s in range(3):
                ii, jj = i + r - 1, j + s - 1
                if 0 <= ii < H and 0 <= jj < W:
                    patch[0, r, s] = x[bi, ii, jj]
        acc = oref.conv_fwd_acc(patch, w, pad=0)[0, 0, 0]          # one output pixel, all channels
        worst = max(worst, int(np.abs(acc).max()))
        want = _psr_vec(oref, acc, bp, 7)
        if relu:
            want = np.maximum(want, 0)
        assert np.array_equal(y[bi, i, j].astype(np.int64), want), (bi, i, j)
    assert worst.bit_length() <= b


def test_config4_forward_layers_sampled(niti, oref):
    from paper_2009_13108_b200 import NitiTrainer
    net = config_net(4)
    x, labels, weights = make_net_inputs(net)
    tr = NitiTrainer(niti, net, weights)
    tr.load_batch(x, labels)
    tr.forward()
    niti.check()
    rng = np.random.default_rng(7)
    a = x
    wi = 0
    for li, L in enumerate(net.layers):
        out = tr.acts[li].cpu().numpy()
        if L["op"] == "conv":
            b = int(tr.b_fwd[li])
            _check_conv_fwd_samples(oref, a, weights[wi], out, b, L["relu"], rng,
                                    n_samples=12 if L["cin"] > 128 else 24)
            assert int(np.abs(out.astype(np.int16)).max()) <= 127
            wi += 1
        elif L["op"] == "pool":
            # exact on a sampled image
            bi = int(rng.integers(a.shape[0]))
            assert np.array_equal(out[bi:bi + 1], oref.maxpool2_fwd(a[bi:bi + 1]))
        else:
            a2 = a.reshape(a.shape[0], -1)
            want, s, b = oref.linear_fwd(a2, int(tr.s_act[li - 1]) if li else net.s_in, weights[wi],
                                         L["s_w"], L["relu"])
            assert np.array_equal(out, want) and int(tr.b_fwd[li]) == b
            wi += 1
        a = out
    assert niti.tc_launch_count() >= 16


@pytest.mark.parametrize("B,H,W,Ci,Co", [(64, 224, 224, 64, 64), (64, 56, 56, 256, 256),
                                         (64, 14, 14, 512, 512)])
def test_config4_backward_ops_sampled(niti, oref, B, H, W, Ci, Co):
    rng = np.random.default_rng(B + H + Ci)
    x = rng.integers(-127, 128, size=(B, H, W, Ci), dtype=np.int8)
    x = np.maximum(x, 0)                                             # a ReLU output feeds the layer
    e = rng.integers(-127, 128, size=(B, H, W, Co), dtype=np.int8)
    w = rng.integers(-127, 128, size=(Co, 3, 3, Ci), dtype=np.int8)
    dev = niti.device
    xt, et, wt = (torch.from_numpy(v).to(dev) for v in (x, e, w))
    # ---- dgrad with the ReLU mask: e_prev[b,i,j,:] from the 3x3 patch of e
    ep, b_e = niti.conv_dgrad(et, wt, (H, W), relu_mask_src=xt)
    niti.check()
    ep = ep.cpu().numpy()
    b = int(b_e)
    bp = max(0, b - 7)
    wflip = np.ascontiguousarray(w[:, ::-1, ::-1, :].transpose(3, 1, 2, 0))   # [Ci][3][3][Co]
    worst = 0
    pts = [(0, 0, 0), (B - 1, H - 1, W - 1)] + [(int(rng.integers(B)), int(rng.integers(H)),
                                                 int(rng.integers(W))) for _ in range(10)]
    for (bi, i, j) in pts:
        patch = np.zeros((1, 3, 3, Co), np.int8)
        for r in range(3):
            for s in range(3):
                ii, jj = i + r - 1, j + s - 1
                if 0 <= ii < H and 0 <= jj < W:
                    patch[0, r, s] = e[bi, ii, jj]
        acc = oref.conv_fwd_acc(patch, wflip, pad=0)[0, 0, 0]
        worst = max(worst, int(np.abs(acc).max()))
        want = np.where(x[bi, i, j] > 0, _psr_vec(oref, acc, bp, 7), 0)
        assert np.array_equal(ep[bi, i, j].astype(np.int64), want), (bi, i, j)
    assert worst.bit_length() <= b
    assert 64 <= int(np.abs(niti.conv_dgrad(et, wt, (H, W))[0].cpu().numpy().astype(np.int16)).max()) <= 127
    # ---- wgrad: sampled entries, each a sum over every pixel
    g, b_g = niti.conv_wgrad(xt, et, m_u=5)
    niti.check()
    g = g.cpu().numpy()
    bg = int(b_g)
    bpg = max(0, bg - 5)
    assert 16 <= int(np.abs(g.astype(np.int16)).max()) <= 31
    e64 = e.astype(np.int64)
    entries = [(0, 0, 0, 0), (Co - 1, 2, 2, Ci - 1)] + [(int(rng.integers(Co)), int(rng.integers(3)),
                                                        int(rng.integers(3)), int(rng.integers(Ci)))
                                                       for _ in range(6)]
    for (co, r, s, ci) in entries:
        xs = np.zeros((B, H, W), np.int64)
        i0, i1 = max(0, 1 - r), min(H, H + 1 - r)
        j0, j1 = max(0, 1 - s), min(W, W + 1 - s)
        xs[:, i0:i1, j0:j1] = x[:, i0 + r - 1:i1 + r - 1, j0 + s - 1:j1 + s - 1, ci]
        acc = int((e64[:, :, :, co] * xs).sum())
        assert abs(acc).bit_length() <= bg
        assert int(g[co, r, s, ci]) == oref.psr(acc, bpg, 5), (co, r, s, ci)


def _full_step_vs_oracle(niti, net, steps):
    from oracle import OracleNetState, oracle_train_step
    from paper_2009_13108_b200 import NitiTrainer
    x, labels, weights = make_net_inputs(net)
    st = OracleNetState([w.copy() for w in weights])
    tr = NitiTrainer(niti, net, weights)
    tr.load_batch(x, labels)
    for step in range(steps):
        rec = oracle_train_step(net, x, labels, st)
        tr.step()
        niti.check()
        assert int(tr.n_correct) == rec["n_correct"]
        assert [int(b) for b in tr.b_fwd] == rec["b_fwd"]
        for k, (wg, wo) in enumerate(zip(tr.weights, st.weights)):
            assert np.array_equal(wg.cpu().numpy(), wo), (step, k)


def test_config2_full_size_steps(niti):
    _full_step_vs_oracle(niti, config_net(2), steps=3)


def test_config3_full_size_step(niti):
    _full_step_vs_oracle(niti, config_net(3), steps=1)
