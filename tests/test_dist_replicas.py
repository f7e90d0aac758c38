"""The N > 1 paths with two gloo ranks on CPU: the benchmark's replicas (max-over-ranks timing, whole-job
throughput, per-rank seeds) and the reducer that the exact data-parallel mode hands its max / sum
words to (the two-rank run of the kernels themselves is tests/test_gpu_dp.py)."""
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


def _reducer_worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2009_13108_b200.api import REDUCE_MAX_U32, REDUCE_MAX_U64, REDUCE_SUM_I32, dist_reducer
    reduce = dist_reducer()
    # the three quantities the exact data-parallel mode combines, as the library hands them over:
    # slices of a byte workspace viewed as int32 / int64
    ws = torch.zeros(256 + 64, dtype=torch.uint8)
    m32 = ws[0:4].view(torch.int32)
    m64 = ws[8:16].view(torch.int64)
    acc = ws[256:256 + 16].view(torch.int32)
    m32[0] = 1000 + 7 * rank
    m64[0] = (1 << 40) + (3 - rank)
    acc.copy_(torch.tensor([5, -6, 7 * (rank + 1), -2147483000 * rank], dtype=torch.int32))
    reduce(m32, REDUCE_MAX_U32)
    reduce(m64, REDUCE_MAX_U64)
    reduce(acc, REDUCE_SUM_I32)
    # the sharded weight-gradient path: reduce-scatter of int32 sums (each rank only needs its own
    # slice afterwards), then all-gather of the int8 slices every rank produced from them
    from paper_2009_13108_b200.api import ALLGATHER_I8, REDUCE_SCATTER_SUM_I32
    g32 = torch.arange(8, dtype=torch.int32) * (rank + 1)
    reduce(g32, REDUCE_SCATTER_SUM_I32)
    mine = g32[rank * 4:(rank + 1) * 4].tolist()
    g8 = torch.full((8,), -1, dtype=torch.int8)
    g8[rank * 4:(rank + 1) * 4] = torch.tensor([10 * rank + i for i in range(4)], dtype=torch.int8)
    reduce(g8, ALLGATHER_I8)
    q.put((rank, int(m32[0]), int(m64[0]), acc.tolist(), mine, g8.tolist()))
    dist.barrier()
    dist.destroy_process_group()


def test_the_data_parallel_reducer_combines_max_and_sum_over_two_gloo_ranks():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_reducer_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, m32, m64, acc, mine, g8 in res:             # the same on every rank
        assert m32 == 1007
        assert m64 == (1 << 40) + 3
        assert acc == [10, -12, 21, -2147483000]
        assert mine == [3 * i for i in range(rank * 4, rank * 4 + 4)]      # sums over ranks 1x + 2x
        assert g8 == [0, 1, 2, 3, 10, 11, 12, 13]


def test_launch_ranks_starts_one_process_per_rank_on_localhost(tmp_path):
    """`bench.py --gpus N` without an external launcher starts its N ranks through this helper."""
    from paper_2009_13108_b200.dist_util import launch_ranks
    worker = os.path.join(os.path.dirname(os.path.abspath(__file__)), "_spawn_worker.py")
    rc = launch_ranks([worker, str(tmp_path)], 2, timeout=300)
    assert rc == 0
    rows = sorted(open(os.path.join(tmp_path, "rank%d.txt" % r)).read().split() for r in range(2))
    assert rows == [["0", "2", "0", "127.0.0.1", "3"], ["1", "2", "1", "127.0.0.1", "3"]]
