"""The N > 1 path of the benchmark is replicas only: its plumbing (max-over-ranks timing, whole-job
throughput, per-rank seeds) is covered here with two gloo ranks on CPU."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2009_13108_b200.dist_util import aggregate_throughput, max_over_ranks, rank_seed


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from synth import config_net, make_net_inputs
    net = config_net(0)
    net.seed = rank_seed(net.seed, rank)
    x, labels, _ = make_net_inputs(net)
    ms_local = [10.0 + rank, 20.0 - rank]               # rank 1 is slower on the first, faster on the second
    ms = max_over_ranks(ms_local)
    q.put((rank, ms, int(x.astype(int).sum()), aggregate_throughput(net.batch, ms[0], world)))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_reduce_timing_and_draw_distinct_batches():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, ms0, sum0, thr0), (r1, ms1, sum1, thr1) = res
    assert ms0 == ms1 == [11.0, 20.0]                    # maximum over ranks, same on every rank
    assert sum0 != sum1                                  # different seeds, different batches
    assert thr0 == thr1 == 64 * 2 / 0.011                # whole-job images per second


def test_single_process_is_the_identity():
    assert max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
    assert aggregate_throughput(64, 5.0, 1) == 12800.0
