"""Bit-exact parity of every C-ABI op against the CPU oracle on seeded inputs (GPU only).

Sizes are chosen so the oracle finishes in seconds while the tensor-core engine still sees
several tiles, ragged tails, every operand layout (K-major / MN-major, 32/64/128-byte swizzle),
split contractions and the fallback engine."""
from ctypes import c_uint32 as C_uint32

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


def _i8(rng, shape):
    return rng.integers(-127, 128, size=shape, dtype=np.int8)


def _T(niti, a):
    return torch.from_numpy(np.ascontiguousarray(a)).to(niti.device)


def _eq(t, want):
    got = t.cpu().numpy()
    assert got.shape == want.shape
    assert np.array_equal(got, want), "mismatch at %s" % np.argwhere(got != want)[:4].tolist()


FC_SHAPES = [(64, 256, 784), (64, 10, 256), (300, 520, 384), (128, 256, 128), (130, 70, 100),
             (257, 300, 96), (1, 32, 32), (64, 1000, 512), (512, 384, 2048)]


@pytest.mark.parametrize("engine", [0, 1, 2, 3, 4])
@pytest.mark.parametrize("M,N,K", FC_SHAPES)
def test_linear_fwd(niti, oref, M, N, K, engine):
    rng = np.random.default_rng(M * 7 + N * 3 + K)
    a, w = _i8(rng, (M, K)), _i8(rng, (N, K))
    niti.set_engine(engine)
    try:
        for relu, mode in [(False, 0), (True, 0), (False, 1)]:
            want, s, b = oref.linear_fwd(a, -7, w, -10, relu, mode)
            out, s_out, b_out = niti.linear_fwd(_T(niti, a), niti.scalar(-7), _T(niti, w),
                                                niti.scalar(-10), relu=relu, round_mode=mode)
            _eq(out, want)
            assert (int(s_out), int(b_out)) == (s, b)
    finally:
        niti.set_engine(0)
    niti.check()


# Many rows, a contraction of one or two k-blocks and a narrow output: the engine batches several
# 128-row tiles per work item (the shape of the gathered RGB first layer).  M is not a multiple of
# the batch (4 x 128 rows) nor of 128, so the last item has missing tiles and a ragged one.
@pytest.mark.parametrize("M,N,K", [(152000 + 77, 64, 32), (152000 + 300, 48, 200), (152000 + 513, 128, 96),
                                   (152000, 20, 32)])
def test_linear_fwd_row_batched(niti, oref, M, N, K):
    rng = np.random.default_rng(M + N + K)
    a, w = _i8(rng, (M, K)), _i8(rng, (N, K))
    for relu, mode in [(True, 0), (False, 1)]:
        want, s, b = oref.linear_fwd(a, -7, w, -10, relu, mode)
        out, s_out, b_out = niti.linear_fwd(_T(niti, a), niti.scalar(-7), _T(niti, w),
                                            niti.scalar(-10), relu=relu, round_mode=mode)
        _eq(out, want)
        assert (int(s_out), int(b_out)) == (s, b)
    niti.check()


@pytest.mark.parametrize("engine", [0, 1, 2, 3, 4])
@pytest.mark.parametrize("M,N,K", FC_SHAPES[:7] + [(640, 256, 512)])
def test_linear_bwd(niti, oref, M, N, K, engine):
    rng = np.random.default_rng(M * 5 + N * 11 + K)
    a, w, e = _i8(rng, (M, K)), _i8(rng, (N, K)), _i8(rng, (M, N))
    mask = np.maximum(a, 0)
    niti.set_engine(engine)
    try:
        for m_u, use_mask in [(5, True), (3, False)]:
            we, wg, be, bg = oref.linear_bwd(a, e, w, True, mask if use_mask else None, m_u)
            ep, g, b_e, b_g = niti.linear_bwd(_T(niti, a), _T(niti, e), _T(niti, w), True,
                                              _T(niti, mask) if use_mask else None, m_u=m_u)
            _eq(ep, we)
            _eq(g, wg)
            assert (int(b_e), int(b_g)) == (be, bg)
            assert int(g.abs().max()) <= 2 ** m_u - 1
        # first layer: no error to propagate
        _, wg, _, bg = oref.linear_bwd(a, e, w, False, None, 5)
        ep, g, _, b_g = niti.linear_bwd(_T(niti, a), _T(niti, e), _T(niti, w), False)
        assert ep is None
        _eq(g, wg)
    finally:
        niti.set_engine(0)
    niti.check()


CONV_SHAPES = [(2, 8, 8, 3, 16), (2, 16, 16, 64, 64), (4, 8, 8, 128, 256), (8, 4, 4, 256, 128),
               (2, 32, 32, 32, 64), (3, 28, 28, 1, 32), (2, 28, 28, 32, 64), (32, 2, 2, 512, 512),
               (1, 56, 56, 64, 128), (2, 12, 20, 96, 160), (2, 24, 40, 128, 128), (1, 64, 48, 64, 64),
               (2, 18, 10, 128, 64), (3, 30, 22, 32, 96),
               # more than 256 output channels: with CTA pairs (engine 3) the tile is 192 columns wide
               # and the last column tile narrower
               (4, 8, 8, 64, 320),
               # RGB first layers: staged gather (W % 4 == 0; one with more pixel groups than threads)
               # and the generic gather (W % 4 != 0)
               (3, 20, 36, 3, 32), (1, 6, 520, 3, 16), (2, 9, 10, 3, 16),
               # more few-channel first layers (gathered taps): RGB and single-channel, several widths
               (2, 32, 32, 3, 64), (4, 32, 16, 1, 32), (8, 64, 48, 3, 16), (3, 16, 48, 3, 32), (2, 32, 16, 1, 32)]


@pytest.mark.parametrize("engine", [0, 1, 2, 3, 4, 5])
@pytest.mark.parametrize("B,H,W,Ci,Co", CONV_SHAPES)
def test_conv_ops(niti, oref, B, H, W, Ci, Co, engine):
    rng = np.random.default_rng(B + H * 3 + W * 5 + Ci * 7 + Co * 11)
    x, w, e = _i8(rng, (B, H, W, Ci)), _i8(rng, (Co, 3, 3, Ci)), _i8(rng, (B, H, W, Co))
    xm = np.maximum(x, 0)
    niti.set_engine(engine)
    try:
        wy, s, b = oref.conv_fwd(x, -7, w, -9, 1, True)
        y, s_y, b_y = niti.conv_fwd(_T(niti, x), niti.scalar(-7), _T(niti, w), niti.scalar(-9),
                                    relu=True)
        _eq(y, wy)
        assert (int(s_y), int(b_y)) == (s, b)
        wd, bd = oref.conv_dgrad(e, w, (H, W), 1, xm)
        ep, b_e = niti.conv_dgrad(_T(niti, e), _T(niti, w), (H, W), relu_mask_src=_T(niti, xm))
        _eq(ep, wd)
        assert int(b_e) == bd
        wg, bg = oref.conv_wgrad(x, e, (3, 3), 1, 5)
        g, b_g = niti.conv_wgrad(_T(niti, x), _T(niti, e))
        _eq(g, wg)
        assert int(b_g) == bg
    finally:
        niti.set_engine(0)
    niti.check()


UPDATE_CONV_SHAPES = [(2, 16, 16, 64, 64), (4, 8, 8, 128, 256), (3, 20, 36, 3, 32), (2, 12, 20, 96, 160),
                      (1, 6, 5, 16, 32)]


@pytest.mark.parametrize("engine", [0, 1, 4])
@pytest.mark.parametrize("B,H,W,Ci,Co", UPDATE_CONV_SHAPES)
def test_conv_wgrad_update(niti, oref, B, H, W, Ci, Co, engine):
    """Weight gradient fused with the update = the oracle's wgrad followed by its weight update."""
    rng = np.random.default_rng(B + H * 3 + W * 5 + Ci * 7 + Co * 13)
    x, e = _i8(rng, (B, H, W, Ci)), _i8(rng, (B, H, W, Co))
    w = rng.integers(-127, 128, size=(Co, 3, 3, Ci), dtype=np.int8)       # extremes: the clamp is exercised
    niti.set_engine(engine)
    try:
        for m_u in (5, 7):
            wg, bg = oref.conv_wgrad(x, e, (3, 3), 1, m_u)
            want = oref.sgd_update(w, wg)
            wt = _T(niti, w.copy())
            got, b_g = niti.conv_wgrad_update(_T(niti, x), _T(niti, e), wt, m_u=m_u)
            assert got.data_ptr() == wt.data_ptr()
            _eq(wt, want)
            assert int(b_g) == bg
    finally:
        niti.set_engine(0)
    niti.check()


@pytest.mark.parametrize("engine", [0, 1])
@pytest.mark.parametrize("M,N,K", [(64, 256, 784), (32, 10, 256), (128, 1000, 512), (300, 384, 640)])
def test_linear_bwd_update(niti, oref, M, N, K, engine):
    rng = np.random.default_rng(M + 3 * N + 7 * K)
    a, e = _i8(rng, (M, K)), _i8(rng, (M, N))
    w = rng.integers(-127, 128, size=(N, K), dtype=np.int8)
    am = np.maximum(a, 0)
    niti.set_engine(engine)
    try:
        we, wg, be, bg = oref.linear_bwd(am, e, w, True, am, 5)
        want_w = oref.sgd_update(w, wg)
        wt = _T(niti, w.copy())
        e_prev, b_e, b_g = niti.linear_bwd_update(_T(niti, am), _T(niti, e), wt, relu_mask_src=_T(niti, am))
        _eq(e_prev, we)                      # from the weights before the update
        _eq(wt, want_w)
        assert (int(b_e), int(b_g)) == (be, bg)
        # without the error of the layer below
        wt2 = _T(niti, w.copy())
        none, _, b_g2 = niti.linear_bwd_update(_T(niti, am), _T(niti, e), wt2, need_e_prev=False)
        assert none is None and int(b_g2) == bg
        _eq(wt2, want_w)
    finally:
        niti.set_engine(0)
    niti.check()


@pytest.mark.parametrize("M,N,K,launches", [(64, 1024, 2048, 1), (96, 768, 1056, 1), (64, 2048, 4096, 3)])
def test_linear_bwd_update_inside_the_multiply(niti, oref, M, N, K, launches):
    """A fully connected weight gradient whose every CTA has one tile rounds with the exact shift in the
    multiply's own epilogue, which then also subtracts from the weights (Section 3.3): one launch, no
    update kernel, the gradient never stored.  Larger ones keep the speculative pass, its follow-up and
    the update kernel.  Weights at +-127 with gradients of either sign exercise the clamp."""
    rng = np.random.default_rng(M + N + K)
    a, e = np.maximum(_i8(rng, (M, K)), 0), _i8(rng, (M, N))
    w = rng.integers(-127, 128, size=(N, K), dtype=np.int8)
    w[::3, ::5] = 127
    w[1::3, 1::5] = -127
    _, wg, _, bg = oref.linear_bwd(a, e, w, False, None, 5)
    want_w = oref.sgd_update(w, wg)
    wt = _T(niti, w.copy())
    at, et = _T(niti, a), _T(niti, e)
    niti.linear_bwd_update(at, et, _T(niti, w.copy()), need_e_prev=False)      # sizes the workspace
    niti.begin_step()
    redo0, n0, t0 = niti.redo_count(), niti.launch_count(), niti.tc_launch_count()
    none, _, b_g = niti.linear_bwd_update(at, et, wt, need_e_prev=False)
    assert niti.tc_launch_count() - t0 == min(launches, 2)
    assert niti.launch_count() - n0 == launches           # 1: nothing but the multiply itself
    assert niti.redo_count() == redo0
    assert none is None and int(b_g) == bg
    _eq(wt, want_w)
    niti.check()


def test_two_contexts_on_one_device(niti, oref):
    """The shared-memory limit of a kernel belongs to the device: a second context whose first launch
    needs little must not lower it under a context that launches with more."""
    from paper_2009_13108_b200 import Niti
    rng = np.random.default_rng(5)
    big = (_i8(rng, (512, 1024)), _i8(rng, (512, 1024)))             # 8 stages of 32 KB
    small = (_i8(rng, (16, 32)), _i8(rng, (32, 32)))                 # two small stages
    want_big = oref.linear_fwd(big[0], -7, big[1], -9, False)
    want_small = oref.linear_fwd(small[0], -7, small[1], -9, False)
    sa, sw = niti.scalar(-7), niti.scalar(-9)
    _eq(niti.linear_fwd(_T(niti, big[0]), sa, _T(niti, big[1]), sw)[0], want_big[0])
    other = Niti(0)
    _eq(other.linear_fwd(_T(other, small[0]), other.scalar(-7), _T(other, small[1]), other.scalar(-9))[0], want_small[0])
    _eq(niti.linear_fwd(_T(niti, big[0]), sa, _T(niti, big[1]), sw)[0], want_big[0])
    _eq(other.linear_fwd(_T(other, big[0]), other.scalar(-7), _T(other, big[1]), other.scalar(-9))[0], want_big[0])
    other.check()
    other.close()
    niti.check()


def test_header_slots_of_a_step(oref):
    """niti_begin_step clears 64 header slots at once and the following calls take one each; the 65th
    and later calls, and calls after the workspace has been replaced by a larger one, clear their own
    header again.  The results never change, and no call of the first 64 enqueues a memset."""
    from paper_2009_13108_b200 import Niti
    niti = Niti(0)                                               # (its own, small workspace)
    rng = np.random.default_rng(64)
    M, N, K = 48, 96, 160
    a, w = _i8(rng, (M, K)), _i8(rng, (N, K))
    want, s_want, b_want = oref.linear_fwd(a, -7, w, -9, True)
    at, wt = _T(niti, a), _T(niti, w)
    sa, sw = niti.scalar(-7), niti.scalar(-9)
    niti.linear_fwd(at, sa, wt, sw, relu=True)                   # sizes the workspace
    niti.begin_step()
    per_call = []
    for i in range(70):
        n0 = niti.launch_count()
        out, s_out, b_out = niti.linear_fwd(at, sa, wt, sw, relu=True)
        per_call.append(niti.launch_count() - n0)
        _eq(out, want)
        assert (int(s_out), int(b_out)) == (s_want, b_want), i
    assert len(set(per_call[:64])) == 1 and per_call[64] == per_call[0] + 1 and per_call[69] == per_call[64]
    # a larger workspace replaces the prepared one: its headers were never cleared by begin_step
    niti.begin_step()
    M2, N2, K2 = 256, 512, 384
    a2, w2 = _i8(rng, (M2, K2)), _i8(rng, (N2, K2))
    want2, s2, b2 = oref.linear_fwd(a2, -7, w2, -9, False)
    out2, s_out2, b_out2 = niti.linear_fwd(_T(niti, a2), sa, _T(niti, w2), sw)
    _eq(out2, want2)
    assert (int(s_out2), int(b_out2)) == (s2, b2)
    out, s_out, b_out = niti.linear_fwd(at, sa, wt, sw, relu=True)
    _eq(out, want)
    niti.check()
    niti.close()


def test_outputs_and_masks_aligned_to_16_but_not_32_bytes(niti, oref):
    """The epilogue's whole-chunk loop needs 32-byte aligned rows; 16-byte aligned tensors take the
    general loop (16-byte stores) and must give the same bytes."""
    import torch
    rng = np.random.default_rng(77)
    B, H, W, Ci, Co = 2, 16, 24, 64, 64
    x, w, e = _i8(rng, (B, H, W, Ci)), _i8(rng, (Co, 3, 3, Ci)), _i8(rng, (B, H, W, Co))
    xm = np.maximum(x, 0)

    def off16(shape):
        n = int(np.prod(shape))
        buf = torch.empty(n + 64, dtype=torch.int8, device=niti.device)
        skew = (16 - buf.data_ptr() % 32) % 32          # 16 mod 32
        return buf[skew:skew + n].view(shape)

    wy, s, b = oref.conv_fwd(x, -7, w, -9, 1, True)
    y = off16((B, H, W, Co))
    assert y.data_ptr() % 32 == 16
    niti.conv_fwd(_T(niti, x), niti.scalar(-7), _T(niti, w), niti.scalar(-9), y=y, relu=True)
    _eq(y, wy)
    wd, bd = oref.conv_dgrad(e, w, (H, W), 1, xm)
    mask = off16((B, H, W, Ci))
    mask.copy_(_T(niti, xm))
    ep, b_e = niti.conv_dgrad(_T(niti, e), _T(niti, w), (H, W), relu_mask_src=mask)
    _eq(ep, wd)
    assert int(b_e) == bd
    a, wl = _i8(rng, (300, 256)), _i8(rng, (192, 256))
    want, s2, b2 = oref.linear_fwd(a, -7, wl, -9, True)
    out = off16((300, 192))
    niti.linear_fwd(_T(niti, a), niti.scalar(-7), _T(niti, wl), niti.scalar(-9), out=out, relu=True)
    _eq(out, want)
    niti.check()


def test_tensor_core_engine_is_the_one_that_runs(niti):
    rng = np.random.default_rng(1)
    before = niti.tc_launch_count()
    a, w = _T(niti, _i8(rng, (256, 512))), _T(niti, _i8(rng, (256, 512)))
    niti.linear_fwd(a, niti.scalar(-7), w, niti.scalar(-10))
    x, wc = _T(niti, _i8(rng, (2, 16, 16, 64))), _T(niti, _i8(rng, (64, 3, 3, 64)))
    e = _T(niti, _i8(rng, (2, 16, 16, 64)))
    niti.conv_fwd(x, niti.scalar(-7), wc, niti.scalar(-9))
    niti.conv_dgrad(e, wc, (16, 16))
    niti.conv_wgrad(x, e)
    niti.linear_bwd(a, _T(niti, _i8(rng, (256, 256))), w)
    assert niti.tc_launch_count() - before >= 6
    niti.check()


@pytest.mark.parametrize("engine", [0, 2, 3])
def test_speculative_shift_is_corrected(niti, oref, engine):
    """The fused epilogue rounds with the bit-width of the first tile of every CTA and redoes the
    multiply when the whole tensor needs a larger shift: here only the last rows are large."""
    rng = np.random.default_rng(77)
    M, N, K = 128 * 400, 64, 128
    a = rng.integers(-3, 4, size=(M, K), dtype=np.int8)
    a[-5:] = rng.integers(100, 128, size=(5, K), dtype=np.int8)
    w = rng.integers(64, 128, size=(N, K), dtype=np.int8)
    want, s, b = oref.linear_fwd(a, -7, w, -10, True)
    niti.set_engine(engine)
    try:
        redo0 = niti.redo_count()
        out, s_out, b_out = niti.linear_fwd(_T(niti, a), niti.scalar(-7), _T(niti, w),
                                            niti.scalar(-10), relu=True)
        _eq(out, want)
        assert (int(s_out), int(b_out)) == (s, b)
        assert niti.redo_count() > redo0, "the second pass did not run: the case no longer tests it"
        # and the mirrored case through the masked dgrad epilogue
        e = rng.integers(-2, 3, size=(M, N), dtype=np.int8)
        e[-3:] = 127
        mask = rng.integers(-5, 6, size=(M, K), dtype=np.int8)
        we, wg, be, bg = oref.linear_bwd(a, e, w, True, mask, 5)
        ep, g, b_e, b_g = niti.linear_bwd(_T(niti, a), _T(niti, e), _T(niti, w), True, _T(niti, mask))
        _eq(ep, we)
        _eq(g, wg)
        assert (int(b_e), int(b_g)) == (be, bg)
    finally:
        niti.set_engine(0)
    niti.check()


def test_speculative_estimate_learns_what_it_missed_at_a_call_site(niti, oref):
    """A call site (recognised by the address of its bit-width scalar) whose extremes sit outside the
    sampled first tiles mispredicts twice (a miss that repeats is taken as systematic), then no more;
    when the data changes the estimate follows after one more recomputation.  Every result is exact."""
    M, N, K = 128 * 400, 64, 128
    w = np.full((N, K), 100, np.int8)
    base = np.where(np.arange(M) % 2 == 0, 5, 6).astype(np.int8)[:, None].repeat(K, 1)   # sums up to 76800: 17 bits
    tail = base.copy()
    tail[-5:] = 11                                                                       # 140800: 18 bits
    wt = _T(niti, w)
    s_a, s_w = niti.scalar(-7), niti.scalar(-10)
    out = torch.empty((M, N), dtype=torch.int8, device=niti.device)
    s_out, b_out = niti.scalar(), niti.scalar(-1)
    redo = []
    for a, bits in ((tail, 18), (tail, 18), (tail, 18), (tail, 18), (base, 17), (base, 17)):
        want, s, b = oref.linear_fwd(a, -7, w, -10, True)
        assert b == bits
        r0 = niti.redo_count()
        niti.linear_fwd(_T(niti, a), s_a, wt, s_w, out=out, s_out=s_out, b_out=b_out, relu=True)
        _eq(out, want)
        assert (int(s_out), int(b_out)) == (s, b)
        redo.append(niti.redo_count() - r0)
    assert redo == [1, 1, 0, 0, 1, 0], redo
    niti.check()


def test_speculative_shift_is_corrected_in_conv_and_row_batched_modes(niti, oref):
    """Same for the resident-weights convolution (small channel counts) and for the row-batched
    multiply of short contractions: only the end of the tensor is large."""
    rng = np.random.default_rng(78)
    B, H, W, C = 40, 32, 32, 64
    x = rng.integers(-3, 4, size=(B, H, W, C), dtype=np.int8)
    x[-1, -4:, -8:] = rng.integers(100, 128, size=(4, 8, C), dtype=np.int8)   # inside the last 8x16 tile only
    w = rng.integers(64, 128, size=(C, 3, 3, C), dtype=np.int8)
    want, s, b = oref.conv_fwd(x, -7, w, -9, 1, True)
    redo0 = niti.redo_count()
    y, s_y, b_y = niti.conv_fwd(_T(niti, x), niti.scalar(-7), _T(niti, w), niti.scalar(-9), relu=True)
    _eq(y, want)
    assert (int(s_y), int(b_y)) == (s, b)
    assert niti.redo_count() > redo0
    M, N, K = 152000 + 130, 64, 32
    a = rng.integers(-3, 4, size=(M, K), dtype=np.int8)
    a[-5:] = rng.integers(100, 128, size=(5, K), dtype=np.int8)
    wf = rng.integers(64, 128, size=(N, K), dtype=np.int8)
    want, s, b = oref.linear_fwd(a, -7, wf, -10, False)
    redo0 = niti.redo_count()
    out, s_out, b_out = niti.linear_fwd(_T(niti, a), niti.scalar(-7), _T(niti, wf), niti.scalar(-10))
    _eq(out, want)
    assert (int(s_out), int(b_out)) == (s, b)
    assert niti.redo_count() > redo0
    niti.check()


@pytest.mark.parametrize("Ci,Co", [(64, 64), (64, 128)])
def test_conv_resident_weights_many_tiles(niti, oref, Ci, Co):
    """Several tiles per CTA in the resident-weights mode (693 8x16 pixel tiles, an odd count, ragged
    in W and H): stage and accumulator rings wrap, contiguous tile ranges differ in length."""
    rng = np.random.default_rng(Ci + Co)
    B, H, W = 7, 141, 85
    x, w, e = _i8(rng, (B, H, W, Ci)), _i8(rng, (Co, 3, 3, Ci)), _i8(rng, (B, H, W, Co))
    wy, s, b = oref.conv_fwd(x, -7, w, -9, 1, True)
    y, s_y, b_y = niti.conv_fwd(_T(niti, x), niti.scalar(-7), _T(niti, w), niti.scalar(-9), relu=True)
    _eq(y, wy)
    assert (int(s_y), int(b_y)) == (s, b)
    xm = np.maximum(x, 0)
    wd, bd = oref.conv_dgrad(e, w, (H, W), 1, xm)
    ep, b_e = niti.conv_dgrad(_T(niti, e), _T(niti, w), (H, W), relu_mask_src=_T(niti, xm))
    _eq(ep, wd)
    assert int(b_e) == bd
    niti.check()


def test_general_taps_and_padding_use_the_fallback(niti, oref):
    rng = np.random.default_rng(2)
    x, w = _i8(rng, (2, 9, 9, 4)), _i8(rng, (6, 5, 5, 4))
    for pad in (0, 2):
        wy, s, b = oref.conv_fwd(x, -7, w, -9, pad, False)
        y, s_y, b_y = niti.conv_fwd(_T(niti, x), niti.scalar(-7), _T(niti, w), niti.scalar(-9),
                                    pad=pad)
        _eq(y, wy)
        e = _i8(rng, wy.shape)
        wd, _ = oref.conv_dgrad(e, w, (9, 9), pad)
        _eq(niti.conv_dgrad(_T(niti, e), _T(niti, w), (9, 9), pad=pad)[0], wd)
        wg, _ = oref.conv_wgrad(x, e, (5, 5), pad, 5)
        _eq(niti.conv_wgrad(_T(niti, x), _T(niti, e), (5, 5), pad=pad)[0], wg)
    niti.check()


@pytest.mark.parametrize("engine", [0, 2, 3])
@pytest.mark.parametrize("R,pad", [(5, 2), (7, 3), (1, 0)])
@pytest.mark.parametrize("B,H,W,Ci,Co", [(2, 16, 16, 32, 64), (8, 12, 20, 64, 128), (3, 8, 16, 128, 32),
                                         (2, 24, 40, 64, 64)])
def test_large_and_pointwise_filters_on_the_tensor_cores(niti, oref, B, H, W, Ci, Co, R, pad, engine):
    """5x5, 7x7 (the paper's LeNet / AlexNet filter sizes, Section 4) and 1x1 convolutions with "same"
    geometry and at least 32 channels run on the tcgen05 kernel: forward, error and weight gradient
    against the oracle, and the tensor-core launch counter must move for each of them."""
    rng = np.random.default_rng(B + H * 3 + W * 5 + Ci * 7 + Co * 11 + R)
    x, w, e = _i8(rng, (B, H, W, Ci)), _i8(rng, (Co, R, R, Ci)), _i8(rng, (B, H, W, Co))
    xm = np.maximum(x, 0)
    niti.set_engine(engine)
    try:
        n0 = niti.tc_launch_count()
        wy, s, b = oref.conv_fwd(x, -7, w, -9, pad, True)
        y, s_y, b_y = niti.conv_fwd(_T(niti, x), niti.scalar(-7), _T(niti, w), niti.scalar(-9), pad=pad, relu=True)
        _eq(y, wy)
        assert (int(s_y), int(b_y)) == (s, b)
        n1 = niti.tc_launch_count()
        wd, bd = oref.conv_dgrad(e, w, (H, W), pad, xm)
        ep, b_e = niti.conv_dgrad(_T(niti, e), _T(niti, w), (H, W), relu_mask_src=_T(niti, xm), pad=pad)
        _eq(ep, wd)
        assert int(b_e) == bd
        n2 = niti.tc_launch_count()
        wg, bg = oref.conv_wgrad(x, e, (R, R), pad, 5)
        g, b_g = niti.conv_wgrad(_T(niti, x), _T(niti, e), (R, R), pad=pad)
        _eq(g, wg)
        assert int(b_g) == bg
        n3 = niti.tc_launch_count()
        if engine != 3:       # (3 = paired CTAs only: a test switch that falls back where pairs do not apply)
            assert n1 > n0 and n2 > n1 and n3 > n2, "a multiply fell back to the CUDA-core engine"
    finally:
        niti.set_engine(0)
    niti.check()


@pytest.mark.parametrize("engine", [0, 1])
@pytest.mark.parametrize("Ci,Co", [(64, 64), (32, 128)])
def test_accumulator_range_is_flagged_where_the_oracle_reports_an_overflow(niti, oref, Ci, Co, engine):
    """int32 accumulators (Section 3.2): the weight gradient contracts over batch x pixels.  With
    constant +127 operands the centre tap sums pixels * 16129: 120000 pixels stay below 2^31 (result
    equal to the oracle's, no flag), 140800 pixels exceed it (the int64 oracle reports the overflow
    and the device status word must carry NITI_DEV_ACC_RANGE)."""
    from oracle.ref import ERR_OVERFLOW, OracleError
    from paper_2009_13108_b200.api import NitiError
    niti.set_engine(engine)
    try:
        for H, overflow in ((300, False), (352, True)):
            x = np.full((1, H, 400, Ci), 127, np.int8)
            e = np.full((1, H, 400, Co), 127, np.int8)
            g, b_g = niti.conv_wgrad(_T(niti, x), _T(niti, e))
            if overflow:
                with pytest.raises(OracleError) as oerr:
                    oref.conv_wgrad(x, e, (3, 3), 1, 5)
                assert oerr.value.code == ERR_OVERFLOW
                with pytest.raises(NitiError):
                    niti.check()
                st = C_uint32()
                assert niti.lib.niti_check(niti.h, niti._stream(), st) == 0     # the word was cleared
            else:
                wg, bg = oref.conv_wgrad(x, e, (3, 3), 1, 5)
                _eq(g, wg)
                assert int(b_g) == bg
                assert niti.check() == 0
        # fully connected weight gradient: contraction over the batch
        for M, overflow in ((120000, False), (140000, True)):
            a = np.full((M, 64), 127, np.int8)
            e = np.full((M, 32), 127, np.int8)
            w = np.zeros((32, 64), np.int8)
            _, g, _, b_g = niti.linear_bwd(_T(niti, a), _T(niti, e), _T(niti, w), need_e_prev=False)
            if overflow:
                with pytest.raises(OracleError):
                    oref.linear_bwd(a, e, w, False)
                with pytest.raises(NitiError) as gerr:
                    niti.check()
                assert "0x10" in str(gerr.value)
            else:
                _, wg, _, bg = oref.linear_bwd(a, e, w, False)
                _eq(g, wg)
                assert int(b_g) == bg and niti.check() == 0
    finally:
        niti.set_engine(0)


STRIDED_SHAPES = [
    # B, H, W, Ci, Co, R, pad, stride
    (2, 23, 23, 3, 16, 11, 2, 4),      # the geometry of the paper's AlexNet first layer (11 x 11, stride 4), RGB input
    (4, 16, 16, 32, 64, 3, 1, 2),      # tensor cores: element stride 2
    (2, 32, 32, 64, 128, 5, 2, 2),
    (8, 24, 24, 128, 64, 3, 1, 3),
    (8, 33, 31, 64, 64, 3, 0, 2),      # odd sizes, no padding: rows the windows never reach
    (3, 28, 28, 1, 32, 5, 0, 1),       # LeNet's 5 x 5 first layer without padding (gathered taps)
    (8, 20, 20, 32, 64, 5, 0, 1),      # "valid" convolution on the tensor cores: output smaller than input
    (8, 12, 12, 64, 32, 3, 3, 1),      # padding larger than (R - 1) / 2: output larger than input
]


@pytest.mark.parametrize("engine", [0, 1])
@pytest.mark.parametrize("B,H,W,Ci,Co,R,pad,stride", STRIDED_SHAPES)
def test_strided_and_unpadded_convolutions(niti, oref, B, H, W, Ci, Co, R, pad, stride, engine):
    """Strides other than 1 and paddings other than (R - 1) / 2, forward / error / weight gradient,
    against the oracle; with at least 32 channels on both sides the forward pass and the weight gradient
    must run on the tensor cores (the error of a strided layer is the CUDA-core engine's)."""
    rng = np.random.default_rng(B + H * 3 + W * 5 + Ci * 7 + Co * 11 + R + 13 * stride)
    x, w = _i8(rng, (B, H, W, Ci)), _i8(rng, (Co, R, R, Ci))
    Ho, Wo = oref.conv_out_hw(H, W, R, R, pad, stride)
    e = _i8(rng, (B, Ho, Wo, Co))
    xm = np.maximum(x, 0)
    niti.set_engine(engine)
    try:
        n0 = niti.tc_launch_count()
        wy, s, b = oref.conv_fwd(x, -7, w, -9, pad, True, stride=stride)
        y, s_y, b_y = niti.conv_fwd(_T(niti, x), niti.scalar(-7), _T(niti, w), niti.scalar(-9), pad=pad,
                                    relu=True, stride=stride)
        _eq(y, wy)
        assert (int(s_y), int(b_y)) == (s, b)
        n1 = niti.tc_launch_count()
        wd, bd = oref.conv_dgrad(e, w, (H, W), pad, xm, stride=stride)
        ep, b_e = niti.conv_dgrad(_T(niti, e), _T(niti, w), (H, W), relu_mask_src=_T(niti, xm), pad=pad,
                                  stride=stride)
        _eq(ep, wd)
        assert int(b_e) == bd
        n2 = niti.tc_launch_count()
        wg, bg = oref.conv_wgrad(x, e, (R, R), pad, 5, stride=stride)
        g, b_g = niti.conv_wgrad(_T(niti, x), _T(niti, e), (R, R), pad=pad, stride=stride)
        _eq(g, wg)
        assert int(b_g) == bg
        n3 = niti.tc_launch_count()
        if engine == 0 and Ci >= 32 and Co >= 32:
            assert n1 > n0 and n3 > n2, "forward / weight gradient fell back to the CUDA-core engine"
            assert (n2 > n1) == (stride == 1)
    finally:
        niti.set_engine(0)
    niti.check()


POOL_SHAPES = [(2, 32, 32, 64, 64), (3, 28, 36, 64, 128), (2, 16, 16, 256, 256), (8, 8, 8, 128, 512),
               (16, 4, 4, 512, 512), (32, 2, 2, 512, 512), (1, 64, 64, 256, 64), (2, 12, 20, 96, 160),
               (2, 6, 10, 32, 48), (3, 20, 36, 3, 32), (2, 16, 64, 128, 128), (1, 18, 26, 64, 64),
               (2, 34, 22, 128, 128), (2, 32, 32, 3, 64), (4, 32, 16, 1, 32)]


@pytest.mark.parametrize("engine", [0, 1, 2, 3, 4, 5])
@pytest.mark.parametrize("B,H,W,Ci,Co", POOL_SHAPES)
def test_conv_fwd_pool(niti, oref, B, H, W, Ci, Co, engine):
    """Convolution + ReLU + 2 x 2 max-pool in one call: both outputs equal the oracle's convolution
    followed by its pooling, whether the tensor-core epilogue pools (windows inside a warp: 8 x 16 pixel
    tiles, narrow pixel boxes, ragged tiles) or the pooling kernel runs afterwards (wide pixel boxes, 48
    output channels, the gathered RGB layer, the other engines)."""
    rng = np.random.default_rng(B + H * 3 + W * 5 + Ci * 7 + Co * 11)
    x, w = _i8(rng, (B, H, W, Ci)), _i8(rng, (Co, 3, 3, Ci))
    wy, s, b = oref.conv_fwd(x, -7, w, -9, 1, True)
    wp = oref.maxpool2_fwd(wy)
    niti.set_engine(engine)
    try:
        y, yp, s_y, b_y = niti.conv_fwd_pool(_T(niti, x), niti.scalar(-7), _T(niti, w), niti.scalar(-9))
        _eq(y, wy)
        _eq(yp, wp)
        assert (int(s_y), int(b_y)) == (s, b)
    finally:
        niti.set_engine(0)
    niti.check()


def test_conv_fwd_pool_after_a_wrong_speculative_shift(niti, oref):
    """The pooled tensor is rewritten with the full-resolution one when the first pass rounded with too
    small a shift (only the end of the tensor is large)."""
    rng = np.random.default_rng(79)
    B, H, W, C = 40, 32, 32, 64
    x = rng.integers(-3, 4, size=(B, H, W, C), dtype=np.int8)
    x[-1, -4:, -8:] = rng.integers(100, 128, size=(4, 8, C), dtype=np.int8)
    w = rng.integers(64, 128, size=(C, 3, 3, C), dtype=np.int8)
    wy, s, b = oref.conv_fwd(x, -7, w, -9, 1, True)
    redo0 = niti.redo_count()
    y, yp, s_y, b_y = niti.conv_fwd_pool(_T(niti, x), niti.scalar(-7), _T(niti, w), niti.scalar(-9))
    _eq(y, wy)
    _eq(yp, oref.maxpool2_fwd(wy))
    assert (int(s_y), int(b_y)) == (s, b) and niti.redo_count() > redo0
    niti.check()


def test_saturation_and_zero_tensor(niti, oref):
    # all-zero accumulators: b = 0, output zero, exponent = s_a + s_w
    a = np.zeros((32, 64), np.int8)
    w = _i8(np.random.default_rng(3), (32, 64))
    out, s_out, b_out = niti.linear_fwd(_T(niti, a), niti.scalar(-7), _T(niti, w), niti.scalar(-3))
    assert int(out.abs().max()) == 0 and int(b_out) == 0 and int(s_out) == -10
    # an accumulator whose integer part is already 127 and whose fraction asks for +1
    a = np.zeros((32, 64), np.int8)
    w = np.zeros((32, 64), np.int8)
    a[0, :4] = [127, 127, 1, 0]
    w[0, :4] = [127, 127, 127, 0]      # 32385: 15 bits, bp = 8, q = 126 ... generic check below
    a[1, :3] = [127, 127, 127]
    w[1, :3] = [86, 0, 0]
    want, s, b = oref.linear_fwd(a, 0, w, 0)
    out, s_out, b_out = niti.linear_fwd(_T(niti, a), niti.scalar(0), _T(niti, w), niti.scalar(0))
    _eq(out, want)
    assert int(out.max()) <= 127 and int(out.min()) >= -127


@pytest.mark.parametrize("s_a", [-22, -9, -7, -6, -4, 0, 24])
@pytest.mark.parametrize("B,N", [(64, 10), (64, 1000), (7, 33), (256, 10), (9, 64), (3, 4096)])
def test_int_xent(niti, oref, s_a, B, N):
    rng = np.random.default_rng(1000 + s_a + B + N)
    a = _i8(rng, (B, N))
    labels = rng.integers(0, N, size=B).astype(np.int32)
    for mode in (0, 1):
        want, b, nc = oref.int_xent(a, s_a, labels, mode)
        e, b_e, n_correct = niti.int_xent(_T(niti, a), niti.scalar(s_a), _T(niti, labels),
                                          round_mode=mode)
        _eq(e, want)
        assert (int(b_e), int(n_correct)) == (b, nc)
    niti.check()


@pytest.mark.parametrize("s_a", [-22, -8, -7, -6, -5, -3, 0, 9, 16, 24])
def test_int_xent_packed_rows(niti, oref, s_a):
    """Rows of whole 32-bit words take the packed-byte path: ties of the maximum before and after
    the label, labels in every byte position of a word, constant rows, narrow and wide logit ranges."""
    rng = np.random.default_rng(5000 + s_a)
    B, N = 48, 64 * 5
    a = _i8(rng, (B, N))
    labels = rng.integers(0, N, size=B).astype(np.int32)
    a[0] = 0                                              # constant row
    a[1] = rng.integers(-2, 3, size=N)                    # narrow range
    a[2] = -127; a[2, 17] = 127; labels[2] = 17           # one dominant logit, on the label
    a[3] = -127; a[3, 18] = 127; labels[3] = 200          # ... off the label
    for k in range(4):                                    # label in every byte position, tie before it
        r = 4 + k
        labels[r] = 100 + k
        a[r, 100 + k] = 90; a[r, 3] = 90; a[r] = np.minimum(a[r], 90)
    for k in range(4):                                    # tie after the label only: the label is the first arg-max
        r = 8 + k
        labels[r] = 40 + k
        a[r] = np.minimum(a[r], 77); a[r, 40 + k] = 77; a[r, 300] = 77; a[r, :40 + k] = np.minimum(a[r, :40 + k], 76)
    labels[12], labels[13] = 0, N - 1                     # first and last element
    for mode in (0, 1):
        want, b, nc = oref.int_xent(a, s_a, labels, mode)
        e, b_e, n_correct = niti.int_xent(_T(niti, a), niti.scalar(s_a), _T(niti, labels), round_mode=mode)
        _eq(e, want)
        assert (int(b_e), int(n_correct)) == (b, nc)
    niti.check()


@pytest.mark.parametrize("s_a", [-22, -9, -7, -6, -4, -2, 0, 3, 9, 24])
@pytest.mark.parametrize("B,N", [(1024, 64), (1500, 1000), (4096, 128)])
def test_int_xent_many_rows_use_precomputed_tables(niti, oref, s_a, B, N):
    """From 1024 rows on, the T and rounded-T tables are computed once per call (one line per
    possible offset p) and the rows copy their line: same bytes as the oracle, rows with narrow,
    constant and extreme logits included."""
    rng = np.random.default_rng(9000 + s_a + B + N)
    a = _i8(rng, (B, N))
    labels = rng.integers(0, N, size=B).astype(np.int32)
    a[0] = 0
    a[1] = rng.integers(-2, 3, size=N)
    a[2] = -127; a[2, 5] = 127; labels[2] = 5
    a[3] = -127; a[3, 6] = 127; labels[3] = 7
    a[4] = 127
    a[5] = -128 + (np.arange(N) % 3 == 0)
    a[6:70] = np.clip(a[6:70] // 16, -8, 7)               # few distinct values: every threshold line gets used
    for mode in (0, 1):
        want, b, nc = oref.int_xent(a, s_a, labels, mode)
        e, b_e, n_correct = niti.int_xent(_T(niti, a), niti.scalar(s_a), _T(niti, labels), round_mode=mode)
        _eq(e, want)
        assert (int(b_e), int(n_correct)) == (b, nc)
    niti.check()


def test_int_xent_flags_bad_domain(niti):
    from paper_2009_13108_b200 import NitiError
    a = torch.zeros((4, 8), dtype=torch.int8, device=niti.device)
    labels = torch.zeros(4, dtype=torch.int32, device=niti.device)
    niti.int_xent(a, niti.scalar(30), labels)
    with pytest.raises(NitiError):
        niti.check()
    labels[2] = 8
    niti.int_xent(a, niti.scalar(-4), labels)
    with pytest.raises(NitiError):
        niti.check()
    assert niti.check() == 0


@pytest.mark.parametrize("n", [1, 15, 16, 17, 4096, 100003, 1 << 22])
def test_sgd_update_and_relu(niti, oref, n):
    rng = np.random.default_rng(n)
    w, g = _i8(rng, n), _i8(rng, n)
    wt = _T(niti, w)
    niti.int_sgd_update(wt, _T(niti, g))
    _eq(wt, oref.sgd_update(w, g))
    x, e = _i8(rng, n), _i8(rng, n)
    y = niti.relu_fwd(_T(niti, x))
    _eq(y, oref.relu_fwd(x))
    _eq(niti.relu_bwd(y, _T(niti, e)), oref.relu_bwd(oref.relu_fwd(x), e))


@pytest.mark.parametrize("B,H,W,C", [(2, 4, 6, 16), (3, 8, 8, 5), (2, 28, 28, 64), (1, 2, 2, 1),
                                     (4, 6, 10, 48)])
def test_maxpool(niti, oref, B, H, W, C):
    rng = np.random.default_rng(B + H + W + C)
    x = np.maximum(rng.integers(-40, 40, size=(B, H, W, C)), 0).astype(np.int8)   # many ties
    e = _i8(rng, (B, H // 2, W // 2, C))
    y = niti.maxpool2_fwd(_T(niti, x))
    _eq(y, oref.maxpool2_fwd(x))
    _eq(niti.maxpool2_bwd(_T(niti, x), _T(niti, e), relu=False), oref.maxpool2_bwd(x, e))
    _eq(niti.maxpool2_bwd(_T(niti, x), _T(niti, e), relu=True),
        oref.relu_bwd(x, oref.maxpool2_bwd(x, e)))
    xs = _i8(rng, (B, H, W, C))
    _eq(niti.maxpool2_bwd(_T(niti, xs), _T(niti, e)), oref.maxpool2_bwd(xs, e))


@pytest.mark.parametrize("B,H,W,C", [(2, 8, 8, 16), (3, 6, 10, 64), (1, 28, 28, 32), (2, 4, 4, 512)])
def test_maxpool_with_recorded_routing(niti, oref, B, H, W, C):
    """Forward records position and positivity of each window's first maximum; backward uses only
    the codes and the error.  Few distinct values: many ties; negative maxima: the ReLU gate."""
    rng = np.random.default_rng(B + H + W + C)
    for lo, hi in ((-3, 4), (-127, 128), (-5, 1)):
        x = rng.integers(lo, hi, size=(B, H, W, C), dtype=np.int8)
        e = _i8(rng, (B, H // 2, W // 2, C))
        y, idx = niti.maxpool2_fwd_idx(_T(niti, x))
        _eq(y, oref.maxpool2_fwd(x))
        assert tuple(idx.shape) == (B, H // 2, W // 2, C // 2)
        routed = oref.maxpool2_bwd(x, e)
        _eq(niti.maxpool2_bwd_idx(_T(niti, e), idx, x.shape, relu=False), routed)
        _eq(niti.maxpool2_bwd_idx(_T(niti, e), idx, x.shape, relu=True), oref.relu_bwd(x, routed))
    niti.check()


def test_argument_errors(niti):
    from paper_2009_13108_b200 import NitiError
    a = torch.zeros((4, 32), dtype=torch.int8, device=niti.device)
    with pytest.raises(NitiError) as ei:
        niti.linear_bwd(a, a, a, m_u=9)
    assert ei.value.code == 1
    # too small a workspace is refused
    import ctypes
    rc = niti.lib.niti_linear_fwd(niti.h, None, a.data_ptr(), niti.scalar().data_ptr(), a.data_ptr(),
                                  niti.scalar().data_ptr(), a.data_ptr(), None, None, 4, 4, 32, 0, 0,
                                  niti._ws.data_ptr(), ctypes.c_size_t(16))
    assert rc == 3


def test_bounded_wait_reports_a_timeout_and_the_context_survives(niti, oref):
    """Failure detection without a fault: a wait that nothing satisfies runs out, the device status
    word says so, and the next call works."""
    from paper_2009_13108_b200 import NitiError
    niti.selftest_timeout()
    with pytest.raises(NitiError) as ei:
        niti.check()
    assert ei.value.code == 6 and "0x1" in str(ei.value)
    assert niti.check() == 0
    rng = np.random.default_rng(5)
    a, w = _i8(rng, (128, 256)), _i8(rng, (64, 256))
    want, s, b = oref.linear_fwd(a, -7, w, -10)
    out, s_out, b_out = niti.linear_fwd(_T(niti, a), niti.scalar(-7), _T(niti, w), niti.scalar(-10))
    _eq(out, want)
    niti.check()
