"""Exact data parallelism (niti_set_reduce_hook): two ranks with half of the batch each give, bit for
bit, the weights, bit-widths and hit counts of the oracle on the whole batch.  The ranks are two
processes on the one GPU of the test box, combined through the host (gloo); no kernel of one rank
waits for a kernel of the other."""
import os
import subprocess
import sys

import numpy as np
import pytest

from synth import config_net, make_net_inputs

pytestmark = pytest.mark.gpu
HERE = os.path.dirname(os.path.abspath(__file__))


@pytest.mark.parametrize("cfg,batch,steps", [(0, 16, 2), (2, 16, 2), (3, 8, 1)])
def test_two_ranks_equal_one_process_with_the_whole_batch(tmp_path, cfg, batch, steps):
    from oracle import OracleNetState, oracle_train_step
    world = 2
    store = str(tmp_path / "store")
    out = str(tmp_path / "out")
    procs = [subprocess.Popen([sys.executable, os.path.join(HERE, "_dp_worker.py"), str(r), str(world), store, out,
                               str(cfg), str(batch), str(steps)], stdout=subprocess.PIPE, stderr=subprocess.STDOUT)
             for r in range(world)]
    logs = []
    for p in procs:
        try:
            o, _ = p.communicate(timeout=600)
        except subprocess.TimeoutExpired:
            p.kill()
            o, _ = p.communicate()
        logs.append(o.decode(errors="replace")[-2000:])
    assert all(p.returncode == 0 for p in procs), logs
    net = config_net(cfg, batch=batch)
    x, labels, weights = make_net_inputs(net)
    st = OracleNetState([w.copy() for w in weights])
    got = [np.load(out + ".rank%d.npz" % r) for r in range(world)]
    wl = [i for i, L in enumerate(net.layers) if L["op"] != "pool"]
    for step in range(steps):
        rec = oracle_train_step(net, x, labels, st)
        for g in got:                                    # every rank holds the same state
            assert int(g["hits%d" % step][0]) == rec["n_correct"]
            assert int(g["b_loss%d" % step][0]) == rec["b_loss"]
            assert list(g["b_fwd%d" % step]) == rec["b_fwd"]
            assert [int(g["b_g%d" % step][i]) for i in reversed(wl)] == rec["b_g"]
            assert [int(g["b_e%d" % step][i]) for i in reversed(wl)] == rec["b_e"]
            for k, wo in enumerate(st.weights):
                assert np.array_equal(g["w%d_%d" % (step, k)], wo), (step, k)
