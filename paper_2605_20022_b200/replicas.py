"""Host-side logic of `bench.py --gpus N`: N independent replicas, no data-path collective.

The decode-step path does not shard across GPUs (sequences and kv-heads are independent and the
task fixes one GPU per problem), so more GPUs means more replicas.  The only cross-rank traffic
is the timing protocol: a barrier on both sides of the timed region and a MAX over ranks of the
device-measured times.  This module holds exactly that, so it can run under `gloo` on CPU.
"""
from __future__ import annotations

import os
from typing import List, Optional, Sequence, Tuple


def rank_world() -> Tuple[int, int, int]:
    """(rank, world_size, local_rank) from the torchrun environment; (0, 1, 0) without it."""
    return int(os.environ.get("RANK", 0)), int(os.environ.get("WORLD_SIZE", 1)), int(os.environ.get("LOCAL_RANK", 0))


def init(backend: str):
    """Initialise torch.distributed when WORLD_SIZE > 1; returns the module or None."""
    _, world, _ = rank_world()
    if world <= 1:
        return None
    import torch.distributed as dist
    if not dist.is_initialized():
        dist.init_process_group(backend)
    return dist


def barrier(dist) -> None:
    if dist is not None:
        dist.barrier()


def max_over_ranks(values: Sequence[float], dist, device="cpu") -> List[float]:
    """Elementwise MAX of `values` over all ranks (identity for a single process)."""
    if dist is None:
        return [float(v) for v in values]
    import torch
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.tolist()]


def whole_job_us_per_step(ms_total: float, steps: int, world: int) -> float:
    """`world` replicas each finish `steps` steps in `ms_total`: the job does world*steps steps."""
    return ms_total * 1e3 / (steps * world)


def free_port() -> int:
    import socket
    with socket.socket() as so:
        so.bind(("127.0.0.1", 0))
        return so.getsockname()[1]


def launch_replicas(n: int, script: str, argv: Sequence[str]) -> int:
    """Run `script argv` as `n` ranks on this node (one process per GPU) under torch.distributed.run and return
    its exit code.  Used when the benchmark is started as a plain process with --gpus N > 1 and no rank
    environment; the ranks then find RANK / LOCAL_RANK / WORLD_SIZE / MASTER_* in their environment as usual."""
    import subprocess
    import sys
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(free_port()), script, *argv]
    return subprocess.run(cmd).returncode
