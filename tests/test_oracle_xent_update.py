"""Pins for the integer cross-entropy gradient, the weight update and the int8 support ops."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

import pyref

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def test_log2e_constant():
    # Section 3.5: log2(e) ~ 47274 * 2^-15 (the decimal value; the hex the paper prints beside it
    # differs by 2 and is not used)
    assert round(math.log2(math.e) * 2 ** 15) == 47274


def test_worked_examples(oref):
    for line in open(os.path.join(GOLD, "xent_worked.txt")):
        if not line.strip() or line.startswith("#"):
            continue
        head, a, e32, b, e = [list(map(int, p.split())) for p in line.split("|")]
        s_a, label = head
        arr = np.array([a], np.int8)
        assert oref.xent_acc(arr, s_a, [label]).tolist() == [e32]
        eq, bb, _ = oref.int_xent(arr, s_a, [label])
        assert bb == b[0] and eq.tolist() == [e]


@pytest.mark.parametrize("s_a", [-22, -12, -8, -7, -6, -5, -3, 0, 2, 5, 24])
def test_invariants_and_python_transcription(oref, s_a):
    rng = np.random.default_rng(100 + s_a)
    B, N = 9, 12
    a = rng.integers(-127, 128, size=(B, N), dtype=np.int8)
    labels = rng.integers(0, N, size=B).astype(np.int32)
    e32 = oref.xent_acc(a, s_a, labels)
    for r in range(B):
        row = [int(v) for v in e32[r]]
        assert row == pyref.xent_row(a[r], s_a, int(labels[r]))
        assert sum(row) == 0                     # mirror of sum(softmax - onehot) = 0
        for i, v in enumerate(row):
            assert (v <= 0) if i == labels[r] else (v >= 1)


def test_taylor_case_is_the_exact_polynomial(oref):
    for s_a in (-7, -9, -15):
        a = np.array([[127, -127, 0, 1, -1, 64, -77]], np.int8)
        N = a.shape[1]
        e32 = oref.xent_acc(a, s_a, [0])[0]
        scale = 2 ** (1 - 2 * s_a)
        # off-label entries are T_i; T_i / 2^(1-2s) = 1 + x + x^2/2 with x = a_i 2^s exactly
        for i in range(1, N):
            x = Fraction(int(a[0, i])) * Fraction(2) ** s_a
            assert Fraction(int(e32[i]), scale) == 1 + x + x * x / 2
            assert abs(float(Fraction(int(e32[i]), scale)) - math.exp(float(x))) < 0.22


def test_shift_case_powers_of_two(oref):
    rng = np.random.default_rng(7)
    for s_a in (-6, -4, -2, 0, 1):
        a = rng.integers(-127, 128, size=(20, 10), dtype=np.int8)
        labels = np.zeros(20, np.int32)
        e32 = oref.xent_acc(a, s_a, labels)
        for r in range(20):
            T = [int(v) for v in e32[r][1:]]                 # off-label entries
            assert all(t in {1 << k for k in range(10)} for t in T)
            # exponent differences follow floor(a 2^s log2 e) to within 1 where not clipped
            xs = [math.floor(int(v) * 2.0 ** s_a * math.log2(math.e)) for v in a[r][1:]]
            mx = max(range(len(T)), key=lambda i: T[i])
            for i, t in enumerate(T):
                if t > 1 and T[mx] > 1:
                    d_int = int(math.log2(T[mx])) - int(math.log2(t))
                    assert abs(d_int - (xs[mx] - xs[i])) <= 1


def test_rank_agreement_with_float_softmax(oref):
    """No error bound is stated in the paper; a loose sanity check only."""
    rng = np.random.default_rng(8)
    a = rng.integers(-127, 128, size=(64, 10), dtype=np.int8)
    labels = rng.integers(0, 10, size=64).astype(np.int32)
    for s_a in (-8, -5, -4):
        e32 = oref.xent_acc(a, s_a, labels).astype(np.float64)
        z = a.astype(np.float64) * 2.0 ** s_a
        p = np.exp(z - z.max(1, keepdims=True))
        p /= p.sum(1, keepdims=True)
        p[np.arange(64), labels] -= 1
        for r in range(64):
            # the label carries the only non-positive entry; the float arg-max over the other
            # classes is (one of) the integer maxima -- power-of-two values tie often
            assert np.argmin(e32[r]) == np.argmin(p[r]) == labels[r]
            off = [i for i in range(10) if i != labels[r]]
            k = off[int(np.argmax(p[r][off]))]
            assert e32[r][k] >= 0.5 * e32[r][off].max()


def test_domain_and_labels(oref):
    a = np.zeros((1, 4), np.int8)
    for s_a in (-23, 25):
        with pytest.raises(oref.OracleError) as ei:
            oref.xent_acc(a, s_a, [0])
        assert ei.value.code == oref.ERR_RANGE
    with pytest.raises(oref.OracleError):
        oref.xent_acc(a, -3, [4])


def test_rounded_loss_gradient_uses_one_shift_for_the_whole_batch(oref):
    rng = np.random.default_rng(9)
    a = rng.integers(-127, 128, size=(16, 10), dtype=np.int8)
    labels = rng.integers(0, 10, size=16).astype(np.int32)
    e, b, nc = oref.int_xent(a, -4, labels)
    q, b2, bp = oref.shift_round(oref.xent_acc(a, -4, labels), 7)
    assert b == b2 and np.array_equal(e, q)
    assert nc == int((a.argmax(1) == labels).sum())


def test_sgd_update(oref):
    w = np.array([127, 127, -127, -127, 0, 5, -5, 100], np.int8)
    g = np.array([-1, 1, 1, -1, 0, 31, -31, -31], np.int8)
    assert oref.sgd_update(w, g).tolist() == [127, 126, -127, -126, 0, -26, 26, 127]
    rng = np.random.default_rng(10)
    w = rng.integers(-127, 128, size=1000, dtype=np.int8)
    g = rng.integers(-127, 128, size=1000, dtype=np.int8)
    u = oref.sgd_update(w, g)
    assert np.array_equal(u, np.clip(w.astype(int) - g.astype(int), -127, 127).astype(np.int8))
    assert u.min() >= -127
    assert np.array_equal(oref.sgd_update(w, np.zeros_like(w)), w)


def test_relu_and_maxpool_against_torch(oref):
    rng = np.random.default_rng(11)
    x = rng.integers(-127, 128, size=(2, 6, 8, 5), dtype=np.int8)
    assert np.array_equal(oref.relu_fwd(x), np.maximum(x, 0))
    e = rng.integers(-127, 128, size=x.shape, dtype=np.int8)
    assert np.array_equal(oref.relu_bwd(np.maximum(x, 0), e), np.where(x > 0, e, 0))
    xt = torch.from_numpy(x.astype(np.float64)).permute(0, 3, 1, 2)
    yt, idx = torch.nn.functional.max_pool2d(xt, 2, return_indices=True)
    y = oref.maxpool2_fwd(x)
    assert np.array_equal(y, yt.permute(0, 2, 3, 1).numpy().astype(np.int8))
    eo = rng.integers(-127, 128, size=y.shape, dtype=np.int8)
    ei = oref.maxpool2_bwd(x, eo)
    assert ei.astype(int).sum() == eo.astype(int).sum()
    # every routed error sits on a maximum of its window
    B, H, W, Cc = x.shape
    for b in range(B):
        for i in range(H // 2):
            for j in range(W // 2):
                for c in range(Cc):
                    win = x[b, 2 * i:2 * i + 2, 2 * j:2 * j + 2, c]
                    got = ei[b, 2 * i:2 * i + 2, 2 * j:2 * j + 2, c]
                    k = int(np.argmax(win.reshape(-1)))      # numpy argmax = first maximum
                    want = np.zeros(4, np.int8)
                    want[k] = eo[b, i, j, c]
                    assert got.reshape(-1).tolist() == want.tolist()


def test_maxpool_tie_goes_to_first(oref):
    x = np.zeros((1, 2, 2, 1), np.int8)
    ei = oref.maxpool2_bwd(x, np.array([[[[9]]]], np.int8))
    assert ei.reshape(-1).tolist() == [9, 0, 0, 0]
    x = np.array([3, 7, 7, 1], np.int8).reshape(1, 2, 2, 1)
    assert oref.maxpool2_bwd(x, np.array([[[[9]]]], np.int8)).reshape(-1).tolist() == [0, 9, 0, 0]
