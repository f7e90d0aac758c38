"""Multi-process plumbing of the benchmark: one process per GPU, replicas only (every rank trains
its own copy on its own batch; the step has no collective on the data path).  Timing is reduced as
the maximum over ranks, throughput is aggregated over ranks."""
from __future__ import annotations

import os

import torch


def rank_world():
    return int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))


def rank_seed(base_seed: int, rank: int) -> int:
    """Every rank draws its own batch and weights."""
    return base_seed + 1000 * rank


def max_over_ranks(values, device="cpu"):
    """Element-wise maximum of a list of floats over all ranks (identity without a process group)."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return [float(v) for v in values]
    t = torch.tensor([float(v) for v in values], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def aggregate_throughput(units_per_rank: float, ms_max: float, world: int) -> float:
    """Whole-job units per second: all ranks processed units_per_rank in ms_max milliseconds."""
    return units_per_rank * world / (ms_max / 1e3)


def free_port() -> int:
    import socket
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def launch_ranks(script_argv, n_ranks: int, extra_env=None, timeout=None) -> int:
    """Starts ``n_ranks`` processes of ``python <script_argv...>`` on this node through
    ``torch.distributed.run`` (one process per GPU, rendezvous on 127.0.0.1, a free port) and waits
    for them; returns the launcher's exit code.  The ranks read RANK / LOCAL_RANK / WORLD_SIZE /
    MASTER_* from their environment, exactly as under an external launcher."""
    import subprocess
    import sys
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(n_ranks),
           "--master-addr", "127.0.0.1", "--master-port", str(free_port())] + list(script_argv)
    env = dict(os.environ)
    env.update(extra_env or {})
    return subprocess.run(cmd, env=env, timeout=timeout).returncode
