"""Pins for the oracle's matrix multiplies and convolutions (CPU only): float64 library
routines (exact below 2^53), exact integer adjoint identities, hand-enumerated tiny cases,
the 1x1-image special case, and an independent padded sliding-window transcription."""
import os

import numpy as np
import pytest
import torch

import pyref

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _i8(rng, shape):
    return rng.integers(-127, 128, size=shape, dtype=np.int8)


@pytest.mark.parametrize("M,N,K", [(1, 1, 1), (3, 5, 7), (17, 10, 33), (64, 48, 200)])
def test_fc_against_float64_matmul(oref, M, N, K):
    rng = np.random.default_rng(M * 1000 + N * 10 + K)
    a, w, e = _i8(rng, (M, K)), _i8(rng, (N, K)), _i8(rng, (M, N))
    af, wf, ef = a.astype(np.float64), w.astype(np.float64), e.astype(np.float64)
    assert np.array_equal(oref.fc_fwd_acc(a, w), (af @ wf.T).astype(np.int64))
    assert np.array_equal(oref.fc_dgrad_acc(e, w), (ef @ wf).astype(np.int64))
    assert np.array_equal(oref.fc_wgrad_acc(a, e), (ef.T @ af).astype(np.int64))


def test_fc_hand_case(oref):
    a = np.array([[1, 2, 3], [-4, 5, -6]], np.int8)
    w = np.array([[7, 8, 9], [1, 0, -1]], np.int8)
    assert oref.fc_fwd_acc(a, w).tolist() == [[50, -2], [-42, 2]]
    e = np.array([[1, -1], [2, 0]], np.int8)
    assert oref.fc_dgrad_acc(e, w).tolist() == [[6, 8, 10], [14, 16, 18]]
    assert oref.fc_wgrad_acc(a, e).tolist() == [[-7, 12, -9], [-1, -2, -3]]


def _torch_conv(x, w, pad):
    xt = torch.from_numpy(x.astype(np.float64)).permute(0, 3, 1, 2)
    wt = torch.from_numpy(w.astype(np.float64)).permute(0, 3, 1, 2)
    y = torch.nn.functional.conv2d(xt, wt, padding=pad)
    return y.permute(0, 2, 3, 1).contiguous().numpy().astype(np.int64)


@pytest.mark.parametrize("B,H,W,Ci,Co,R,pad", [(1, 4, 4, 1, 1, 3, 1), (2, 5, 7, 3, 4, 3, 1),
                                               (2, 6, 6, 8, 5, 3, 0), (1, 8, 8, 2, 3, 5, 2),
                                               (3, 4, 5, 6, 7, 1, 0)])
def test_conv_against_float64_conv2d(oref, B, H, W, Ci, Co, R, pad):
    rng = np.random.default_rng(B + 10 * H + 100 * Ci + 1000 * Co + R)
    x, w = _i8(rng, (B, H, W, Ci)), _i8(rng, (Co, R, R, Ci))
    y = oref.conv_fwd_acc(x, w, pad)
    assert np.array_equal(y, _torch_conv(x, w, pad))
    # transposes via torch autograd-free identities: dgrad = conv_transpose2d, wgrad = conv of
    # x with e as the kernel
    e = _i8(rng, y.shape)
    et = torch.from_numpy(e.astype(np.float64)).permute(0, 3, 1, 2)
    wt = torch.from_numpy(w.astype(np.float64)).permute(0, 3, 1, 2)
    xt = torch.from_numpy(x.astype(np.float64)).permute(0, 3, 1, 2)
    ex = torch.nn.functional.conv_transpose2d(et, wt, padding=pad).permute(0, 2, 3, 1).numpy()
    assert np.array_equal(oref.conv_dgrad_acc(e, w, (H, W), pad), ex.astype(np.int64))
    gw = torch.nn.grad.conv2d_weight(xt, wt.shape, et, padding=pad).permute(0, 2, 3, 1).numpy()
    assert np.array_equal(oref.conv_wgrad_acc(x, e, (R, R), pad), gw.astype(np.int64))


STRIDED = [(1, 7, 7, 1, 1, 3, 1, 2), (2, 9, 8, 3, 4, 3, 1, 2), (1, 23, 23, 3, 5, 11, 2, 4),
           (2, 10, 10, 4, 3, 5, 2, 2), (1, 8, 9, 2, 2, 2, 0, 2), (2, 6, 7, 3, 2, 1, 0, 3)]


@pytest.mark.parametrize("B,H,W,Ci,Co,R,pad,stride", STRIDED)
def test_strided_conv_against_float64_conv2d(oref, B, H, W, Ci, Co, R, pad, stride):
    """Strides other than 1 (the first layer of the paper's AlexNet is 11 x 11 with stride 4, Section 4)
    against torch's float64 conv2d / conv_transpose2d / conv2d_weight (exact below 2^53)."""
    rng = np.random.default_rng(B + 10 * H + 100 * Ci + 1000 * Co + R + 7 * stride)
    x, w = _i8(rng, (B, H, W, Ci)), _i8(rng, (Co, R, R, Ci))
    xt = torch.from_numpy(x.astype(np.float64)).permute(0, 3, 1, 2)
    wt = torch.from_numpy(w.astype(np.float64)).permute(0, 3, 1, 2)
    want = torch.nn.functional.conv2d(xt, wt, padding=pad, stride=stride).permute(0, 2, 3, 1).numpy()
    y = oref.conv_fwd_acc(x, w, pad, stride)
    assert y.shape == want.shape == (B,) + oref.conv_out_hw(H, W, R, R, pad, stride) + (Co,)
    assert np.array_equal(y, want.astype(np.int64))
    e = _i8(rng, y.shape)
    et = torch.from_numpy(e.astype(np.float64)).permute(0, 3, 1, 2)
    # input rows the strided windows never reach get no error: output_padding restores the input size
    Ho, Wo = y.shape[1:3]
    op = (H - ((Ho - 1) * stride - 2 * pad + R), W - ((Wo - 1) * stride - 2 * pad + R))
    ex = torch.nn.functional.conv_transpose2d(et, wt, padding=pad, stride=stride, output_padding=op)
    assert np.array_equal(oref.conv_dgrad_acc(e, w, (H, W), pad, stride),
                          ex.permute(0, 2, 3, 1).numpy().astype(np.int64))
    gw = torch.nn.grad.conv2d_weight(xt, wt.shape, et, padding=pad, stride=stride).permute(0, 2, 3, 1).numpy()
    assert np.array_equal(oref.conv_wgrad_acc(x, e, (R, R), pad, stride), gw.astype(np.int64))
    # exact adjoint identities in integers
    lhs = int((y * e.astype(np.int64)).sum())
    assert lhs == int((oref.conv_dgrad_acc(e, w, (H, W), pad, stride) * x.astype(np.int64)).sum())
    assert lhs == int((oref.conv_wgrad_acc(x, e, (R, R), pad, stride) * w.astype(np.int64)).sum())


def test_strided_conv_hand_case(oref):
    """1-D in effect: x = [1..5] on a 1 x 5 image, taps [1, 10, 100] (1 x 3), pad 1, stride 2.
    Windows are centred on x[0], x[2], x[4]: y = [10*1 + 100*2, 2 + 10*3 + 100*4, 4 + 10*5]."""
    x = np.arange(1, 6, dtype=np.int8).reshape(1, 1, 5, 1)
    w = np.zeros((1, 3, 3, 1), np.int8)
    w[0, 1, :, 0] = [1, 10, 100]
    y = oref.conv_fwd_acc(x, w, 1, 2)
    assert y.shape == (1, 1, 3, 1) and y.reshape(-1).tolist() == [210, 432, 54]
    e = np.array([1, 2, 3], np.int8).reshape(1, 1, 3, 1)
    # ex[j] collects e[i] * w[t] with 2 i + t - 1 == j
    assert oref.conv_dgrad_acc(e, w, (1, 5), 1, 2).reshape(-1).tolist() == [10, 100 + 2, 20, 200 + 3, 30]
    g = oref.conv_wgrad_acc(x, e, (3, 3), 1, 2)
    assert g[0, 1, :, 0].tolist() == [2 * 2 + 3 * 4, 1 + 2 * 3 + 3 * 5, 2 + 2 * 4]
    assert int(np.abs(g[0, 0]).sum()) == 0 and int(np.abs(g[0, 2]).sum()) == 0


def test_weight_gradient_loop_order_does_not_matter(oref):
    """The oracle's weight gradient runs the pixels as outer loops; the same sums with the pixel loops
    innermost (the formula read literally), in pure Python on a small case."""
    rng = np.random.default_rng(21)
    B, H, W, Ci, Co, R, pad, stride = 2, 5, 6, 3, 2, 3, 1, 1
    x, e = _i8(rng, (B, H, W, Ci)), _i8(rng, (B, H, W, Co))
    want = np.zeros((Co, R, R, Ci), np.int64)
    for co in range(Co):
        for r in range(R):
            for t in range(R):
                for ci in range(Ci):
                    s = 0
                    for b in range(B):
                        for i in range(H):
                            for j in range(W):
                                ii, jj = i + r - pad, j + t - pad
                                if 0 <= ii < H and 0 <= jj < W:
                                    s += int(e[b, i, j, co]) * int(x[b, ii, jj, ci])
                    want[co, r, t, ci] = s
    assert np.array_equal(oref.conv_wgrad_acc(x, e, (R, R), pad, stride), want)


def test_conv_adjoint_identities(oref):
    """<fwd(x,w), e> = <x, dgrad(e,w)> = <w, wgrad(x,e)>, exactly, in integers."""
    rng = np.random.default_rng(11)
    for (B, H, W, Ci, Co) in [(2, 5, 6, 3, 4), (1, 3, 3, 1, 2), (3, 8, 4, 5, 1)]:
        x, w = _i8(rng, (B, H, W, Ci)), _i8(rng, (Co, 3, 3, Ci))
        e = _i8(rng, (B, H, W, Co))
        lhs = int((oref.conv_fwd_acc(x, w, 1) * e.astype(np.int64)).sum())
        mid = int((oref.conv_dgrad_acc(e, w, (H, W), 1) * x.astype(np.int64)).sum())
        rhs = int((oref.conv_wgrad_acc(x, e, (3, 3), 1) * w.astype(np.int64)).sum())
        assert lhs == mid == rhs


def test_fc_adjoint_identities(oref):
    rng = np.random.default_rng(12)
    a, w, e = _i8(rng, (6, 9)), _i8(rng, (4, 9)), _i8(rng, (6, 4))
    lhs = int((oref.fc_fwd_acc(a, w) * e.astype(np.int64)).sum())
    assert lhs == int((oref.fc_dgrad_acc(e, w) * a.astype(np.int64)).sum())
    assert lhs == int((oref.fc_wgrad_acc(a, e) * w.astype(np.int64)).sum())


def test_conv_linearity(oref):
    rng = np.random.default_rng(13)
    x1 = rng.integers(-60, 61, size=(1, 4, 5, 2), dtype=np.int8)
    x2 = rng.integers(-60, 61, size=(1, 4, 5, 2), dtype=np.int8)
    w = _i8(rng, (3, 3, 3, 2))
    assert np.array_equal(oref.conv_fwd_acc((x1 + x2).astype(np.int8), w, 1),
                          oref.conv_fwd_acc(x1, w, 1) + oref.conv_fwd_acc(x2, w, 1))


def test_conv_on_1x1_image_is_fc_on_centre_tap(oref):
    rng = np.random.default_rng(14)
    x, w = _i8(rng, (5, 1, 1, 7)), _i8(rng, (4, 3, 3, 7))
    y = oref.conv_fwd_acc(x, w, 1).reshape(5, 4)
    assert np.array_equal(y, oref.fc_fwd_acc(x.reshape(5, 7), np.ascontiguousarray(w[:, 1, 1, :])))


def test_conv_hand_enumerated(oref):
    d = {}
    for line in open(os.path.join(GOLD, "conv_tiny.txt")):
        if line.strip() and not line.startswith("#"):
            k, *v = line.split()
            d[k] = np.array(list(map(int, v)))
    x = d["x"].astype(np.int8).reshape(1, 2, 2, 1)
    w = d["w"].astype(np.int8).reshape(1, 3, 3, 1)
    e = d["e"].astype(np.int8).reshape(1, 2, 2, 1)
    assert oref.conv_fwd_acc(x, w, 1).reshape(-1).tolist() == d["y"].tolist()
    assert oref.conv_dgrad_acc(e, w, (2, 2), 1).reshape(-1).tolist() == d["ex"].tolist()
    assert oref.conv_wgrad_acc(x, e, (3, 3), 1).reshape(-1).tolist() == d["g"].tolist()


def test_conv_against_padded_window_transcription(oref):
    rng = np.random.default_rng(15)
    x, w = _i8(rng, (2, 4, 3, 2)), _i8(rng, (3, 3, 3, 2))
    assert np.array_equal(oref.conv_fwd_acc(x, w, 1), pyref.conv_fwd_padded(x, w, 1))


def test_overflow_is_reported(oref):
    # K * 127^2 > 2^31 needs K > 133144
    K = 140000
    a = np.full((1, K), 127, np.int8)
    w = np.full((1, K), 127, np.int8)
    acc = oref.fc_fwd_acc(a, w)
    assert int(acc[0, 0]) == K * 127 * 127 > 2 ** 31
    with pytest.raises(oref.OracleError) as ei:
        oref.linear_fwd(a, 0, w, 0)
    assert ei.value.code == oref.ERR_OVERFLOW


def test_composed_linear_and_conv_ops(oref):
    """The composed ops are the accumulator followed by shift_round, ReLU / mask last, and the
    exponent is the sum of the operand exponents plus the shift (Algorithm 1 and 2)."""
    rng = np.random.default_rng(16)
    a, w = _i8(rng, (9, 40)), _i8(rng, (6, 40))
    out, s_out, b = oref.linear_fwd(a, -7, w, -10, relu=True)
    q, b2, bp = oref.shift_round(oref.fc_fwd_acc(a, w), 7)
    assert b == b2 and s_out == -17 + bp and np.array_equal(out, np.maximum(q, 0))
    e = _i8(rng, (9, 6))
    mask = np.maximum(a, 0)
    e_prev, g, b_e, b_g = oref.linear_bwd(a, e, w, True, mask, 5)
    qe, be2, _ = oref.shift_round(oref.fc_dgrad_acc(e, w), 7)
    qg, bg2, _ = oref.shift_round(oref.fc_wgrad_acc(a, e), 5)
    assert (b_e, b_g) == (be2, bg2)
    assert np.array_equal(e_prev, np.where(mask > 0, qe, 0)) and np.array_equal(g, qg)
    assert np.abs(g.astype(int)).max() <= 31
    x, wc = _i8(rng, (2, 5, 5, 4)), _i8(rng, (3, 3, 3, 4))
    y, s_y, b_y = oref.conv_fwd(x, -7, wc, -8, 1, relu=False)
    q, b2, bp = oref.shift_round(oref.conv_fwd_acc(x, wc, 1), 7)
    assert b_y == b2 and s_y == -15 + bp and np.array_equal(y, q)
    ec = _i8(rng, (2, 5, 5, 3))
    gq, bg = oref.conv_wgrad(x, ec, (3, 3), 1, 4)
    assert np.array_equal(gq, oref.shift_round(oref.conv_wgrad_acc(x, ec), 4)[0])
    assert np.abs(gq.astype(int)).max() <= 15
    eq, be = oref.conv_dgrad(ec, wc, (5, 5), 1)
    assert np.array_equal(eq, oref.shift_round(oref.conv_dgrad_acc(ec, wc, (5, 5)), 7)[0])
