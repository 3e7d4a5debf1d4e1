"""Host-side logic for running the path on several GPUs of one node.

Images are independent, so the path shards over the batch with no data-path collective: every rank packs the
(small) weights itself and convolves its own images.  The only communication is for measurement: a barrier and
two tiny reductions (slowest rank's time, total images).  Works with any torch.distributed backend (NCCL on
GPUs, gloo in the CPU tests).
"""
from __future__ import annotations

from typing import Tuple

import torch
import torch.distributed as dist


def shard_batch(n_total: int, world: int, rank: int) -> Tuple[int, int]:
    """Contiguous slice [start, stop) of a batch of n_total images owned by `rank` (sizes differ by at most 1)."""
    if world < 1 or not (0 <= rank < world) or n_total < 0:
        raise ValueError("invalid sharding arguments")
    base, extra = divmod(n_total, world)
    start = rank * base + min(rank, extra)
    return start, start + base + (1 if rank < extra else 0)


def job_throughput(units_local: float, ms_local: float, device: str = "cpu") -> Tuple[float, float, float]:
    """(units per second of the whole job, slowest rank's milliseconds, total units).

    Every rank passes the units it processed and its own device-measured time; the job's time is the maximum
    over the ranks, its work the sum.  Without an initialised process group the local values are returned."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return units_local / (ms_local * 1e-3), ms_local, units_local
    t = torch.tensor([ms_local], dtype=torch.float64, device=device)
    u = torch.tensor([units_local], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    ms, units = float(t.item()), float(u.item())
    return units / (ms * 1e-3), ms, units
