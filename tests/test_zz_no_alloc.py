"""niti_int_xent_noalloc -- the entry point for callers that may not allocate device memory (no
context, no workspace: its scratch is a fixed array inside the library).  It must give exactly
the bytes of niti_int_xent, on two calls in a row (the shared array keeps the first call's
contents), and refuse inputs beyond its fixed capacity; the same outputs are also compared with the
CPU oracle directly.  Collected last on purpose."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def _case(rng, B, N, dev):
    a = torch.from_numpy(rng.integers(-127, 128, size=(B, N), dtype=np.int8)).to(dev)
    labels = torch.from_numpy(rng.integers(0, N, size=B).astype(np.int32)).to(dev)
    return a, labels


def test_no_alloc_entry_point_matches_the_regular_one(oref):
    from paper_2009_13108_b200 import Niti
    niti = Niti(0)
    dev = niti.device
    rng = np.random.default_rng(2024)
    # two calls in a row on different inputs, shapes and exponents: both loss cases, and the second
    # call must not see anything the first one left in the shared scratch array
    for (B, N, s_a, mode) in [(64, 1000, -4, 0), (37, 10, -9, 1), (256, 10, -5, 0)]:
        a, labels = _case(rng, B, N, dev)
        s = niti.scalar(s_a)
        want_e, want_b, want_nc = niti.int_xent(a, s, labels, round_mode=mode)
        # every buffer is allocated by the caller, before the call
        e = torch.full((B, N), 99, dtype=torch.int8, device=dev)
        b_e, n_correct = niti.scalar(-1), niti.scalar(-1)
        torch.cuda.synchronize()
        before = torch.cuda.memory_allocated(dev)
        rc = niti.int_xent_noalloc(a, s, labels, e, b_e, n_correct, round_mode=mode)
        assert rc == 0
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated(dev) == before
        assert torch.equal(e, want_e)                       # bit-exact: all of this path is integer
        assert int(b_e) == int(want_b) and int(n_correct) == int(want_nc)
        # and against the CPU oracle (Section 3.5), not only against the other CUDA entry point
        ref_e, ref_b, ref_nc = oref.int_xent(a.cpu().numpy(), s_a, labels.cpu().numpy(), mode)
        assert np.array_equal(e.cpu().numpy(), ref_e)
        assert (int(b_e), int(n_correct)) == (ref_b, ref_nc)
    # optional outputs may be omitted
    a, labels = _case(rng, 8, 16, dev)
    e = torch.empty((8, 16), dtype=torch.int8, device=dev)
    assert niti.int_xent_noalloc(a, niti.scalar(-3), labels, e) == 0
    assert torch.equal(e, niti.int_xent(a, niti.scalar(-3), labels)[0])
    niti.check()
    niti.close()


def test_no_alloc_entry_point_rejects_oversize_inputs():
    from paper_2009_13108_b200 import Niti
    niti = Niti(0)
    dev = niti.device
    B, N = 66, 1000                                          # 66000 logits > 65536
    a = torch.zeros((B, N), dtype=torch.int8, device=dev)
    labels = torch.zeros(B, dtype=torch.int32, device=dev)
    e = torch.full((B, N), 7, dtype=torch.int8, device=dev)
    rc = niti.int_xent_noalloc(a, niti.scalar(-4), labels, e)
    assert rc == 8                                           # NITI_ERR_TOO_LARGE
    torch.cuda.synchronize()
    assert int(e.min()) == 7 and int(e.max()) == 7           # nothing was enqueued
    assert niti.int_xent_noalloc(a[:2], niti.scalar(-4), labels[:2], e[:2], round_mode=5) == 1
    niti.close()
