"""Writes the stored expected values of the full-size benchmark configurations.

Calls only ``oracle/`` (the int64 CPU oracle) and ``synth/`` (seeded inputs); nothing here touches
the CUDA library.  Run from the repository root:

    python tests/golden/make_config_goldens.py config4     # ~15 min on 8 cores, ~6 GB
    python tests/golden/make_config_goldens.py config2     # ~5 min on 8 cores

* ``config4_step_sha256.txt``: ONE whole training step (Algorithm 1) of the ImageNet-shaped VGG-16
  stack at 224x224, batch 64: SHA-256 of every activation tensor (post ReLU / pool, as stored), of
  the loss gradient, of every updated weight tensor, and every effective bit-width of the step.
* ``config2_100steps.txt``: 100 consecutive steps of the MNIST-shaped CNN at batch 256 (step t reads
  the mini-batch ``synth.make_step_batch(net, t)``, weights carried from step to step): per step the
  logits' exponent, every bit-width and the hit count; SHA-256 of every weight tensor after steps
  1, 10, 50 and 100.

File format: ``key value`` lines; lists are comma separated; ``#`` starts a comment.
"""
import hashlib
import os
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)
HERE = os.path.dirname(os.path.abspath(__file__))

from oracle import OracleNetState, oracle_train_step, ref  # noqa: E402
from synth import config_net, make_net_inputs, make_step_batch  # noqa: E402


def sha(a) -> str:
    return hashlib.sha256(np.ascontiguousarray(a).tobytes()).hexdigest()


def ints(v) -> str:
    return ",".join(str(int(i)) for i in v)


def scalars(rec, prefix=""):
    return ["%sb_fwd %s" % (prefix, ints(rec["b_fwd"])),
            "%ss_act %s" % (prefix, ints(rec["s_act"])),
            "%sb_loss %d" % (prefix, rec["b_loss"]),
            "%sb_e %s" % (prefix, ints(rec["b_e"])),
            "%sb_g %s" % (prefix, ints(rec["b_g"])),
            "%sn_correct %d" % (prefix, rec["n_correct"])]


def config4():
    net = config_net(4)
    x, labels, weights = make_net_inputs(net)
    st = OracleNetState([w.copy() for w in weights])
    t0 = time.time()
    rec = oracle_train_step(net, x, labels, st, keep_tensors=True)   # raises on an int32 overflow
    out = ["# One training step (Algorithm 1) of config 4 (ImageNet-shaped VGG-16, 224x224, batch 64,",
           "# seed 4, m_u = 5, pseudo-stochastic rounding) computed by the int64 CPU oracle.",
           "# Written by tests/golden/make_config_goldens.py config4 (%d threads, %.0f s)."
           % (ref.n_threads(), time.time() - t0),
           "# b_e and b_g are in the order of the reverse loop (last weight layer first).",
           "input_x %s" % sha(x), "input_labels %s" % sha(labels)]
    out += scalars(rec)
    for i, a in enumerate(rec["tensors"]["act"]):
        out.append("act_%d %s" % (i, sha(a)))
    out.append("e_loss %s" % sha(rec["tensors"]["e_loss"]))
    for i, w in enumerate(st.weights):
        out.append("weight_%d %s" % (i, sha(w)))
    with open(os.path.join(HERE, "config4_step_sha256.txt"), "w") as f:
        f.write("\n".join(out) + "\n")
    print("\n".join(out))


def config2(steps=100):
    net = config_net(2)
    _, _, weights = make_net_inputs(net)
    st = OracleNetState([w.copy() for w in weights])
    out = ["# %d consecutive training steps (Algorithm 1) of config 2 (MNIST-shaped CNN, batch 256, seed 2,"
           % steps,
           "# m_u = 5, pseudo-stochastic rounding) computed by the int64 CPU oracle; step t reads the",
           "# mini-batch synth.make_step_batch(net, t); the weights are carried from step to step.",
           "# Written by tests/golden/make_config_goldens.py config2.",
           "# step <t> <key> <values>: b_e and b_g in the order of the reverse loop.",
           "steps %d" % steps]
    t0 = time.time()
    for t in range(steps):
        x, labels = make_step_batch(net, t)
        try:
            rec = oracle_train_step(net, x, labels, st)
        except ref.OracleError as e:
            # the logits' exponent left the domain of the integer loss (Section 3.5), or an int32
            # accumulator overflowed: the run ends here and the GPU must flag the same step
            out.append("stopped_at_step %d oracle_error %d" % (t, e.code))
            break
        out += scalars(rec, "step %d " % t)
        if t + 1 in (1, 10, 50, steps):
            for i, w in enumerate(st.weights):
                out.append("after_step %d weight_%d %s" % (t + 1, i, sha(w)))
        print("step", t, "s_out", rec["s_out"], "hits", rec["n_correct"], "%.0f s" % (time.time() - t0),
              flush=True)
    with open(os.path.join(HERE, "config2_100steps.txt"), "w") as f:
        f.write("\n".join(out) + "\n")


if __name__ == "__main__":
    which = sys.argv[1] if len(sys.argv) > 1 else "all"
    if which in ("config2", "all"):
        config2()
    if which in ("config4", "all"):
        config4()
