"""Host-side logic of the multi-GPU path.  Samples are independent and the weights are replicated, so the hot path
shards over ranks by samples with no data-path collective; the only exchanges are the bookkeeping ones below (which
rank owns which samples, the job's token count and its slowest rank).  Everything here runs on any torch.distributed
backend: NCCL on GPUs, gloo in the CPU tests."""
from __future__ import annotations

import torch
import torch.distributed as dist


def rank_seed(base_seed: int, rank: int) -> int:
    """Weak scaling: every rank draws its own batch of the workload's shape from its own seed."""
    return int(base_seed) + 1000 * int(rank)


def batch_slice(batch: int, world: int, rank: int) -> slice:
    """Strong scaling: contiguous, balanced slice of the samples owned by `rank` (sizes differ by at most one)."""
    assert 0 <= rank < world and batch >= 0
    q, r = divmod(batch, world)
    lo = rank * q + min(rank, r)
    return slice(lo, lo + q + (1 if rank < r else 0))


def job_throughput(units_local: float, ms_local: float, device="cpu", group=None):
    """Whole-job figures from per-rank ones: (units summed over ranks, time = max over ranks in ms, units per second).
    Without an initialised process group the local values are the job's."""
    if not (dist.is_available() and dist.is_initialized()):
        return float(units_local), float(ms_local), float(units_local) / (float(ms_local) * 1e-3)
    u = torch.tensor([float(units_local)], dtype=torch.float64, device=device)
    t = torch.tensor([float(ms_local)], dtype=torch.float64, device=device)
    dist.all_reduce(u, op=dist.ReduceOp.SUM, group=group)
    dist.all_reduce(t, op=dist.ReduceOp.MAX, group=group)
    return float(u.item()), float(t.item()), float(u.item()) / (float(t.item()) * 1e-3)
