"""Whole training steps (Algorithm 1) on the GPU against the oracle's composition: every weight
tensor, the logits' exponent, every effective bit-width and the hit count must be identical."""
import numpy as np
import pytest
import torch

from synth import config_net, gemm_grad_operands, gemm_operands, make_net_inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def niti():
    from paper_2009_13108_b200 import Niti
    n = Niti(0)
    yield n
    n.check()
    n.close()


def _run_both(niti, net, steps, fused_update=False, pool_codes=False, pool_fused=True):
    from oracle import OracleNetState, oracle_train_step
    from paper_2009_13108_b200 import NitiTrainer
    x, labels, weights = make_net_inputs(net)
    st = OracleNetState([w.copy() for w in weights])
    tr = NitiTrainer(niti, net, weights, fused_update=fused_update, pool_codes=pool_codes, pool_fused=pool_fused)
    tr.load_batch(x, labels)
    for step in range(steps):
        rec = oracle_train_step(net, x, labels, st)
        tr.step()
        niti.check()
        assert int(tr.n_correct) == rec["n_correct"], step
        assert int(tr.b_loss) == rec["b_loss"], step
        got_b = [int(b) for b in tr.b_fwd]
        assert got_b == rec["b_fwd"], step
        wl = [i for i, L in enumerate(net.layers) if L["op"] != "pool"]
        assert [int(tr.b_g[i]) for i in reversed(wl)] == rec["b_g"], step
        assert [int(tr.b_e[i]) for i in reversed(wl)] == rec["b_e"], step
        last = max(i for i, L in enumerate(net.layers) if L["op"] != "pool")
        assert int(tr.s_act[last]) == rec["s_out"], step
        for k, (wg, wo) in enumerate(zip(tr.weights, st.weights)):
            assert np.array_equal(wg.cpu().numpy(), wo), (step, k)
    return tr


def test_nearest_rounding_and_smaller_update_width(niti):
    """The paper's accuracy runs round a and e to nearest and shrink m_u over training."""
    from oracle import OracleNetState, oracle_train_step
    from paper_2009_13108_b200 import NitiTrainer
    for m_u, mode in [(3, 1), (4, 0)]:
        net = config_net(2, batch=16)
        net.m_u = m_u
        x, labels, weights = make_net_inputs(net)
        st = OracleNetState([w.copy() for w in weights])
        tr = NitiTrainer(niti, net, weights, round_mode=mode)
        tr.load_batch(x, labels)
        for _ in range(2):
            rec = oracle_train_step(net, x, labels, st, round_mode=mode)
            tr.step()
            niti.check()
            assert int(tr.n_correct) == rec["n_correct"]
            for wg, wo in zip(tr.weights, st.weights):
                assert np.array_equal(wg.cpu().numpy(), wo)


def test_prefetched_batches_give_the_same_steps(niti):
    """prefetch_batch / commit_batch (copy stream, staging buffers) against load_batch."""
    import torch
    from paper_2009_13108_b200 import NitiTrainer
    net = config_net(2, batch=32)
    x, labels, weights = make_net_inputs(net)
    x2 = np.ascontiguousarray(x[::-1])
    l2 = np.ascontiguousarray(labels[::-1])
    a = NitiTrainer(niti, net, weights)
    b = NitiTrainer(niti, net, weights)
    hx, hl, hx2, hl2 = (torch.from_numpy(v).pin_memory() for v in (x, labels, x2, l2))
    b.prefetch_batch(hx, hl)
    for xb, lb, nx, nl in ((hx, hl, hx2, hl2), (hx2, hl2, hx, hl), (hx, hl, None, None)):
        a.load_batch(xb, lb)
        a.step()
        b.commit_batch()
        if nx is not None:
            b.prefetch_batch(nx, nl)          # overlaps the step below
        b.step()
        niti.check()
        assert int(a.n_correct) == int(b.n_correct)
        for wa, wb in zip(a.weights, b.weights):
            assert torch.equal(wa, wb)


def test_config0_mlp_full_size(niti):
    _run_both(niti, config_net(0), steps=5)


def test_steps_with_the_weight_update_fused_into_the_weight_gradient(niti):
    """Same weights, bit-widths and hit counts as the oracle when the trainer uses the fused calls."""
    _run_both(niti, config_net(0), steps=3, fused_update=True)
    _run_both(niti, config_net(2, batch=32), steps=2, fused_update=True)
    _run_both(niti, config_net(3, batch=8), steps=2, fused_update=True)


def test_steps_with_recorded_pool_routing(niti):
    _run_both(niti, config_net(2, batch=32), steps=2, pool_codes=True)
    _run_both(niti, config_net(3, batch=8), steps=2, pool_codes=True)


def test_config2_mnist_cnn_reduced_batch(niti):
    _run_both(niti, config_net(2, batch=32), steps=3)


def test_config3_cifar_vgg11_reduced_batch(niti):
    tr = _run_both(niti, config_net(3, batch=8), steps=2)
    assert niti.tc_launch_count() > 0


def test_config4_vgg16_shrunk_image(niti):
    # the same 16-layer stack on 32x32 images (the 224x224 original is checked by properties)
    _run_both(niti, config_net(4, batch=4, scale=7), steps=1)


@pytest.mark.parametrize("dist", ["uniform", "gauss"])
@pytest.mark.parametrize("M,N,K", [(256, 256, 256), (1024, 256, 4096), (256, 4096, 1024)])
def test_config1_sweep_small_cases_exact(niti, oref, M, N, K, dist):
    a, w = gemm_operands(M, N, K, dist)
    dev = niti.device
    want, s, b = oref.linear_fwd(a, -7, w, -10)
    out, s_out, b_out = niti.linear_fwd(torch.from_numpy(a).to(dev), niti.scalar(-7),
                                        torch.from_numpy(w).to(dev), niti.scalar(-10))
    assert np.array_equal(out.cpu().numpy(), want) and (int(b_out), int(s_out)) == (b, s)
    # 5-bit gradient variant: g[M][N] = sum_k e[k][m] a[k][n] through the backward entry point
    e, a2 = gemm_grad_operands(M, N, K, dist)
    _, wg, _, bg = oref.linear_bwd(a2, e, np.zeros((M, N), np.int8), False, None, 5)
    _, g, _, b_g = niti.linear_bwd(torch.from_numpy(a2).to(dev), torch.from_numpy(e).to(dev),
                                   torch.zeros((M, N), dtype=torch.int8, device=dev), False, m_u=5)
    assert np.array_equal(g.cpu().numpy(), wg) and int(b_g) == bg
    assert int(g.abs().max()) <= 31
    niti.check()


@pytest.mark.parametrize("M,N,K", [(4096, 4096, 4096), (8192, 8192, 8192), (8192, 256, 8192)])
def test_config1_sweep_full_size_sampled(niti, oref, M, N, K):
    """At the benchmark's sizes the oracle computes sampled outputs one by one.  The effective
    bit-width is pinned by the sampled maxima (lower bound) and by the invariant that the shift
    leaves max |q| in [64, 127]; each sampled output is then rounded by the oracle's scalar rule."""
    a, w = gemm_operands(M, N, K, "uniform")
    at, wt = torch.from_numpy(a).to(niti.device), torch.from_numpy(w).to(niti.device)
    out, s_out, b_out = niti.linear_fwd(at, niti.scalar(-7), wt, niti.scalar(-10))
    niti.check()
    b = int(b_out)
    bp = max(0, b - 7)
    assert int(s_out) == -17 + bp
    mx = int(out.abs().max())
    assert 64 <= mx <= 127
    rng = np.random.default_rng(5)
    rows = rng.integers(0, M, size=24)
    cols = rng.integers(0, N, size=24)
    # whole sampled rows / columns (exercises every column tile and the ragged ends)
    got = out.cpu().numpy()
    for r in rows[:6]:
        acc = oref.fc_fwd_acc(a[r:r + 1], w)[0]
        assert int(np.abs(acc).max()).bit_length() <= b
        want = np.array([oref.psr(int(v), bp, 7) for v in acc], dtype=np.int8)
        assert np.array_equal(got[r], want)
    for c in cols[:6]:
        acc = oref.fc_fwd_acc(a, w[c:c + 1])[:, 0]
        want = np.array([oref.psr(int(v), bp, 7) for v in acc], dtype=np.int8)
        assert np.array_equal(got[:, c], want)


def test_steps_with_separate_pooling_passes(niti):
    """The default forward step pools in the convolution's epilogue; the separate pooling pass gives the
    same steps."""
    _run_both(niti, config_net(3, batch=8), steps=2, pool_fused=False)
    _run_both(niti, config_net(2, batch=16), steps=2, pool_fused=False)
