"""The composed training step (Algorithm 1).  The paper prints no tensor of a step, so the
composition is "parity unpinned" as a whole; it is checked here against an independent
composition written with numpy float64 matmuls / torch convolutions for the sums and the
bit-string rounding of pyref, on tiny nets, tensor by tensor."""
import numpy as np
import torch

import pyref
from oracle import OracleNetState, oracle_train_step
from synth import Net, config_net, make_net_inputs


def _sr(acc, mbits):
    q, b, bp = pyref.shift_round(acc, mbits)
    return q.astype(np.int8), b, bp


def _xent(a, s_a, labels):
    e32 = np.array([pyref.xent_row(a[r], s_a, int(labels[r])) for r in range(a.shape[0])])
    return _sr(e32, 7)[0]


def _conv64(x, w):
    xt = torch.from_numpy(x.astype(np.float64)).permute(0, 3, 1, 2)
    wt = torch.from_numpy(w.astype(np.float64)).permute(0, 3, 1, 2)
    return torch.nn.functional.conv2d(xt, wt, padding=1).permute(0, 2, 3, 1).numpy().astype(np.int64)


def _independent_step(net, x, labels, weights):
    """Forward, loss, backward, update -- written separately from oracle/net.py."""
    ws = [w.copy() for w in weights]
    ins, a, s = [], x, net.s_in
    k = 0
    for L in net.layers:
        ins.append(a)
        if L["op"] == "fc":
            acc = (a.reshape(a.shape[0], -1).astype(np.float64) @ ws[k].astype(np.float64).T)
            a, _, bp = _sr(acc.astype(np.int64), 7)
            s, k = s + L["s_w"] + bp, k + 1
            a = np.maximum(a, 0) if L["relu"] else a
        elif L["op"] == "conv":
            a, _, bp = _sr(_conv64(a, ws[k]), 7)
            s, k = s + L["s_w"] + bp, k + 1
            a = np.maximum(a, 0) if L["relu"] else a
        else:
            B, H, W, C = a.shape
            a = a.reshape(B, H // 2, 2, W // 2, 2, C).max(axis=(2, 4))
    e = _xent(a, s, labels)
    new_ws = list(ws)
    for li in range(len(net.layers) - 1, -1, -1):
        L, a_in = net.layers[li], ins[li]
        if L["op"] == "pool":
            B, H, W, C = a_in.shape
            e = e.reshape(B, H // 2, W // 2, C)
            out = np.zeros_like(a_in)
            for b in range(B):
                for i in range(H // 2):
                    for j in range(W // 2):
                        for c in range(C):
                            win = a_in[b, 2 * i:2 * i + 2, 2 * j:2 * j + 2, c].reshape(-1)
                            kk = int(np.argmax(win))
                            out[b, 2 * i + kk // 2, 2 * j + kk % 2, c] = e[b, i, j, c]
            e = np.where(a_in > 0, out, 0).astype(np.int8)
            continue
        k -= 1
        w = ws[k]
        if L["op"] == "fc":
            a2 = a_in.reshape(a_in.shape[0], -1).astype(np.float64)
            e2 = e.reshape(a2.shape[0], -1).astype(np.float64)
            g, _, _ = _sr((e2.T @ a2).astype(np.int64), net.m_u)
            e_prev = _sr((e2 @ w.astype(np.float64)).astype(np.int64), 7)[0].reshape(a_in.shape)
        else:
            xt = torch.from_numpy(a_in.astype(np.float64)).permute(0, 3, 1, 2)
            et = torch.from_numpy(e.astype(np.float64)).permute(0, 3, 1, 2)
            wt = torch.from_numpy(w.astype(np.float64)).permute(0, 3, 1, 2)
            gw = torch.nn.grad.conv2d_weight(xt, wt.shape, et, padding=1).permute(0, 2, 3, 1)
            g, _, _ = _sr(gw.numpy().astype(np.int64), net.m_u)
            ex = torch.nn.functional.conv_transpose2d(et, wt, padding=1).permute(0, 2, 3, 1)
            e_prev = _sr(ex.numpy().astype(np.int64), 7)[0]
        if li > 0 and net.layers[li - 1]["op"] != "pool" and net.layers[li - 1].get("relu"):
            e_prev = np.where(a_in > 0, e_prev, 0).astype(np.int8)
        new_ws[k] = np.clip(w.astype(int) - g.astype(int), -127, 127).astype(np.int8)
        e = e_prev
    return new_ws, a, s


def _tiny_nets():
    mlp = Net("tiny_mlp", 5, (24,), 4, -7, 100)
    mlp.layers = [{"op": "fc", "k": 24, "n": 16, "relu": True, "s_w": -7},
                  {"op": "fc", "k": 16, "n": 4, "relu": False, "s_w": -7}]
    cnn = Net("tiny_cnn", 3, (4, 4, 2), 3, -7, 101)
    cnn.layers = [{"op": "conv", "cin": 2, "cout": 4, "relu": True, "s_w": -7},
                  {"op": "conv", "cin": 4, "cout": 4, "relu": True, "s_w": -8},
                  {"op": "pool"},
                  {"op": "conv", "cin": 4, "cout": 3, "relu": True, "s_w": -8},
                  {"op": "fc", "k": 12, "n": 3, "relu": False, "s_w": -7}]
    return [mlp, cnn]


def test_step_matches_independent_composition():
    for net in _tiny_nets():
        x, labels, weights = make_net_inputs(net)
        st = OracleNetState([w.copy() for w in weights])
        for step in range(3):
            want_ws, want_logits, want_s = _independent_step(net, x, labels, st.weights)
            rec = oracle_train_step(net, x, labels, st, keep_tensors=True)
            assert np.array_equal(rec["tensors"]["logits"], want_logits)
            assert rec["s_out"] == want_s
            for w_got, w_want in zip(st.weights, want_ws):
                assert np.array_equal(w_got, w_want)
        # the update actually moved the weights
        assert any(not np.array_equal(a, b) for a, b in zip(st.weights, weights))


def test_update_uses_pre_update_weights_for_dgrad():
    """Algorithm 1 computes e(l-1) from w(l) before w(l) is updated."""
    net = _tiny_nets()[0]
    x, labels, weights = make_net_inputs(net)
    st = OracleNetState([w.copy() for w in weights])
    rec = oracle_train_step(net, x, labels, st, keep_tensors=True)
    from oracle import ref
    e_loss = rec["tensors"]["e_loss"]
    a1 = rec["tensors"]["act"][0]
    want = ref.shift_round(ref.fc_dgrad_acc(e_loss, weights[1]), 7)[0]
    want = np.where(a1 > 0, want, 0)
    assert np.array_equal(rec["tensors"]["e"][0], want)


def test_config_shapes():
    n0 = config_net(0)
    assert n0.n_weights() == 784 * 256 + 256 * 256 + 2560 == 268800
    n2 = config_net(2)
    assert n2.n_weights() == 288 + 18432 + 12544 * 128 + 1280
    n3 = config_net(3)
    assert n3.n_weights() == 9222848
    assert n3.layers[-1]["k"] == 512 and n3.macs_per_pass() // 10 ** 8 == 391
    n4 = config_net(4)
    assert n4.layers[-3]["k"] == 25088 and n4.n_weights() // 10 ** 5 == 1383
    assert n4.macs_per_pass() // 10 ** 9 == 990
    assert [L["s_w"] for L in n0.layers] == [-10, -10, -10]
    assert n4.layers[0]["s_w"] == -8 and n4.layers[1]["s_w"] == -10


def test_scaled_config_runs_one_step():
    net = config_net(3, batch=4, scale=1)       # CIFAR-shaped VGG-11, batch cut to 4
    x, labels, weights = make_net_inputs(net)
    st = OracleNetState([w.copy() for w in weights])
    rec = oracle_train_step(net, x, labels, st)
    assert -8 <= rec["s_out"] <= -1 and 0 <= rec["n_correct"] <= 4
    assert all(b <= 31 for b in rec["b_fwd"])
