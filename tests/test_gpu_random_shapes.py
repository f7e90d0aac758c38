"""Seeded random shapes through every multiply of the boundary, against the CPU oracle.

The hand-picked shapes of test_gpu_ops.py aim at known tile, swizzle and wave boundaries; these draw
shapes the planner was not written around (odd row counts, channel counts that are multiples of 16 or 32
but of nothing larger, filters from 1 x 1 to 7 x 7, strides, paddings that leave rows unreached), with
value distributions that move the bit-width around (full range, small magnitudes, a few outliers).
Every case is bit-exact or the test fails; the seeds are fixed, so a failure reproduces."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def niti():
    from paper_2009_13108_b200 import Niti
    n = Niti(0)
    yield n
    n.check()
    n.close()


def _T(niti, a):
    return torch.from_numpy(np.ascontiguousarray(a)).to(niti.device)


def _eq(t, want, what):
    got = t.cpu().numpy()
    assert got.shape == want.shape, what
    assert np.array_equal(got, want), "%s: mismatch at %s" % (what, np.argwhere(got != want)[:4].tolist())


def _draw(rng, shape, kind):
    """int8 tensors of three kinds: full range, small magnitudes, small with a few large outliers."""
    if kind == 0:
        return rng.integers(-127, 128, size=shape, dtype=np.int8)
    a = rng.integers(-6, 7, size=shape, dtype=np.int8)
    if kind == 2:
        flat = a.reshape(-1)
        idx = rng.integers(0, flat.size, size=max(1, flat.size // 4096))
        flat[idx] = rng.integers(100, 128, size=idx.size).astype(np.int8) * rng.choice(np.array([-1, 1], np.int8), idx.size)
    return a


@pytest.mark.parametrize("seed", range(30))
def test_random_fully_connected_layers(niti, oref, seed):
    rng = np.random.default_rng(1000 + seed)
    M = int(rng.choice([1, 7, 33, 64, 100, 128, 257, 384, 777]))
    N = int(rng.choice([10, 16, 48, 96, 100, 256, 272, 520, 1000]))
    K = int(rng.choice([32, 48, 64, 96, 144, 256, 400, 784, 1040]))
    kind = seed % 3
    a, w, e = _draw(rng, (M, K), kind), _draw(rng, (N, K), 0), _draw(rng, (M, N), kind)
    am = np.maximum(a, 0)
    s_a, s_w = int(rng.integers(-9, -3)), int(rng.integers(-11, -6))
    relu, mode, m_u = bool(seed & 1), int(seed % 4 == 3), int(rng.choice([3, 5, 7]))
    tag = "fc M=%d N=%d K=%d kind=%d" % (M, N, K, kind)
    for engine in (0, 1):
        niti.set_engine(engine)
        try:
            want, s, b = oref.linear_fwd(am, s_a, w, s_w, relu, mode)
            out, s_out, b_out = niti.linear_fwd(_T(niti, am), niti.scalar(s_a), _T(niti, w), niti.scalar(s_w),
                                                relu=relu, round_mode=mode)
            _eq(out, want, tag + " fwd")
            assert (int(s_out), int(b_out)) == (s, b), tag
            we, wg, be, bg = oref.linear_bwd(am, e, w, True, am, m_u, mode)
            ep, g, b_e, b_g = niti.linear_bwd(_T(niti, am), _T(niti, e), _T(niti, w), True, _T(niti, am), m_u=m_u,
                                              round_mode=mode)
            _eq(ep, we, tag + " dgrad")
            _eq(g, wg, tag + " wgrad")
            assert (int(b_e), int(b_g)) == (be, bg), tag
            # the fused update gives the weights the separate calls give
            wt = _T(niti, w.copy())
            niti.linear_bwd_update(_T(niti, am), _T(niti, e), wt, relu_mask_src=_T(niti, am), m_u=m_u, round_mode=mode)
            _eq(wt, oref.sgd_update(w, wg), tag + " update")
        finally:
            niti.set_engine(0)
    niti.check()


@pytest.mark.parametrize("seed", range(40))
def test_random_convolutions(niti, oref, seed):
    rng = np.random.default_rng(2000 + seed)
    R = int(rng.choice([1, 3, 3, 3, 5, 7]))
    stride = int(rng.choice([1, 1, 1, 2, 3]))
    pad = int(rng.choice([0, (R - 1) // 2, (R - 1) // 2, R // 2 + 1])) if R > 1 else int(rng.choice([0, 1]))
    Ci = int(rng.choice([1, 3, 16, 32, 48, 64, 96, 128, 160]))
    Co = int(rng.choice([16, 32, 48, 64, 96, 128, 192, 320]))
    H = int(rng.integers(max(R, 5), 30))
    W = int(rng.integers(max(R, 5), 30))
    B = int(rng.choice([1, 2, 3, 5, 8]))
    kind = seed % 3
    Ho, Wo = oref.conv_out_hw(H, W, R, R, pad, stride)
    x, w = _draw(rng, (B, H, W, Ci), kind), _draw(rng, (Co, R, R, Ci), 0)
    e = _draw(rng, (B, Ho, Wo, Co), kind)
    xm = np.maximum(x, 0)
    mode, m_u = int(seed % 5 == 4), int(rng.choice([3, 5]))
    tag = "conv B=%d H=%d W=%d Ci=%d Co=%d R=%d pad=%d stride=%d kind=%d" % (B, H, W, Ci, Co, R, pad, stride, kind)
    for engine in (0, 1):
        niti.set_engine(engine)
        try:
            wy, s, b = oref.conv_fwd(xm, -7, w, -9, pad, True, mode, stride=stride)
            y, s_y, b_y = niti.conv_fwd(_T(niti, xm), niti.scalar(-7), _T(niti, w), niti.scalar(-9), pad=pad,
                                        relu=True, round_mode=mode, stride=stride)
            _eq(y, wy, tag + " fwd")
            assert (int(s_y), int(b_y)) == (s, b), tag
            wd, bd = oref.conv_dgrad(e, w, (H, W), pad, xm, mode, stride=stride)
            ep, b_e = niti.conv_dgrad(_T(niti, e), _T(niti, w), (H, W), relu_mask_src=_T(niti, xm), pad=pad,
                                      round_mode=mode, stride=stride)
            _eq(ep, wd, tag + " dgrad")
            assert int(b_e) == bd, tag
            wg, bg = oref.conv_wgrad(xm, e, (R, R), pad, m_u, mode, stride=stride)
            g, b_g = niti.conv_wgrad(_T(niti, xm), _T(niti, e), (R, R), pad=pad, m_u=m_u, round_mode=mode,
                                     stride=stride)
            _eq(g, wg, tag + " wgrad")
            assert int(b_g) == bg, tag
        finally:
            niti.set_engine(0)
    niti.check()


@pytest.mark.parametrize("seed", range(8))
def test_random_multi_wave_convolutions(niti, oref, seed):
    """Medium 3 x 3 layers with more tiles than SMs (speculative shift over several waves, CTA pairs or
    the resident-weights mode, the fused pooling, the fused update), drawn like the ones above."""
    rng = np.random.default_rng(3000 + seed)
    Ci = int(rng.choice([64, 128, 192, 256]))
    Co = int(rng.choice([64, 128, 256, 320]))
    H = int(rng.choice([20, 28, 36, 44])) + 2 * int(rng.integers(0, 4))
    W = int(rng.choice([24, 32, 40, 56])) + 2 * int(rng.integers(0, 4))
    B = int(rng.choice([8, 12, 16]))
    kind = seed % 3
    x, w = _draw(rng, (B, H, W, Ci), kind), _draw(rng, (Co, 3, 3, Ci), 0)
    e = _draw(rng, (B, H, W, Co), kind)
    xm = np.maximum(x, 0)
    tag = "conv B=%d H=%d W=%d Ci=%d Co=%d kind=%d" % (B, H, W, Ci, Co, kind)
    wy, s, b = oref.conv_fwd(xm, -7, w, -9, 1, True)
    wp = oref.maxpool2_fwd(wy)
    y, y_pool, s_y, b_y = niti.conv_fwd_pool(_T(niti, xm), niti.scalar(-7), _T(niti, w), niti.scalar(-9))
    _eq(y, wy, tag + " fwd")
    _eq(y_pool, wp, tag + " pooled")
    assert (int(s_y), int(b_y)) == (s, b), tag
    wd, bd = oref.conv_dgrad(e, w, (H, W), 1, xm)
    ep, b_e = niti.conv_dgrad(_T(niti, e), _T(niti, w), (H, W), relu_mask_src=_T(niti, xm))
    _eq(ep, wd, tag + " dgrad")
    assert int(b_e) == bd, tag
    wg, bg = oref.conv_wgrad(xm, e, (3, 3), 1, 5)
    wt = _T(niti, w.copy())
    _, b_g = niti.conv_wgrad_update(_T(niti, xm), _T(niti, e), wt)
    _eq(wt, oref.sgd_update(w, wg), tag + " update")
    assert int(b_g) == bg, tag
    niti.check()


DEGENERATE_CONVS = [
    # B, H, W, Ci, Co, R, pad, stride
    (1, 1, 1, 64, 64, 3, 1, 1),        # one pixel: only the centre tap sees data
    (3, 1, 40, 32, 64, 3, 1, 1),       # one image row
    (2, 37, 1, 64, 32, 3, 1, 1),       # one image column
    (1, 2, 2, 128, 128, 3, 1, 1),
    (5, 3, 3, 256, 256, 3, 0, 1),      # unpadded 3 x 3 on 3 x 3: a single output pixel per image
    (1, 7, 7, 512, 512, 7, 0, 1),      # the filter covers the whole image
    (4, 9, 9, 32, 32, 1, 0, 2),        # pointwise, stride 2
    (2, 10, 6, 16, 16, 5, 4, 3),       # padding larger than the data it frames
]


@pytest.mark.parametrize("B,H,W,Ci,Co,R,pad,stride", DEGENERATE_CONVS)
def test_degenerate_convolution_extents(niti, oref, B, H, W, Ci, Co, R, pad, stride):
    rng = np.random.default_rng(B + 3 * H + 5 * W + Ci + Co + R)
    Ho, Wo = oref.conv_out_hw(H, W, R, R, pad, stride)
    x, w, e = _draw(rng, (B, H, W, Ci), 0), _draw(rng, (Co, R, R, Ci), 0), _draw(rng, (B, Ho, Wo, Co), 0)
    xm = np.maximum(x, 0)
    tag = "conv B=%d H=%d W=%d Ci=%d Co=%d R=%d pad=%d stride=%d" % (B, H, W, Ci, Co, R, pad, stride)
    for engine in (0, 1):
        niti.set_engine(engine)
        try:
            wy, s, b = oref.conv_fwd(xm, -7, w, -9, pad, False, stride=stride)
            y, s_y, b_y = niti.conv_fwd(_T(niti, xm), niti.scalar(-7), _T(niti, w), niti.scalar(-9), pad=pad,
                                        stride=stride)
            _eq(y, wy, tag + " fwd")
            assert (int(s_y), int(b_y)) == (s, b), tag
            wd, bd = oref.conv_dgrad(e, w, (H, W), pad, None, stride=stride)
            ep, b_e = niti.conv_dgrad(_T(niti, e), _T(niti, w), (H, W), pad=pad, stride=stride)
            _eq(ep, wd, tag + " dgrad")
            assert int(b_e) == bd, tag
            wg, bg = oref.conv_wgrad(xm, e, (R, R), pad, 5, stride=stride)
            g, b_g = niti.conv_wgrad(_T(niti, xm), _T(niti, e), (R, R), pad=pad, stride=stride)
            _eq(g, wg, tag + " wgrad")
            assert int(b_g) == bg, tag
        finally:
            niti.set_engine(0)
    niti.check()


def test_largest_class_count_of_the_loss(niti, oref):
    """niti_int_xent takes up to 65536 classes; both cases of Section 3.5 on such rows."""
    rng = np.random.default_rng(65536)
    B, N = 3, 65536
    a = _draw(rng, (B, N), 0)
    labels = np.array([0, N - 1, 12345], dtype=np.int32)
    for s_a in (-9, -3):
        want_e, want_b, want_nc = oref.int_xent(a, s_a, labels, 0)
        e, b_e, n_correct = niti.int_xent(_T(niti, a), niti.scalar(s_a), _T(niti, labels))
        _eq(e, want_e, "xent s_a=%d" % s_a)
        assert (int(b_e), int(n_correct)) == (want_b, want_nc)
    niti.check()
