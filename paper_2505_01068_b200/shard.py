"""Host-side logic of the multi-GPU path.  Samples are independent and the weights are replicated, so the hot path
shards over ranks by samples with no data-path collective; the only exchanges are the bookkeeping ones below (which
rank owns which samples, the job's token count and its slowest rank).  Everything here runs on any torch.distributed
backend: NCCL on GPUs, gloo in the CPU tests."""
from __future__ import annotations

import socket

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


def balanced_slices(cost, world: int) -> list[slice]:
    """Strong scaling over samples of unequal length: contiguous slices of the batch whose summed `cost` (e.g. the valid
    tokens of each sample) is as even as contiguous cuts allow.  The first r slices end where the running sum first
    reaches r / world of the total, so every rank's share differs from the ideal by less than one sample's cost; with at
    least `world` samples every slice holds at least one."""
    cost = [float(c) for c in cost]
    n, total = len(cost), sum(cost)
    assert world >= 1
    keep = 1 if n >= world else 0        # samples every slice must get
    cuts, run, i = [0], 0.0, 0
    for r in range(1, world):
        lo, hi = cuts[-1] + keep, n - keep * (world - r)
        while i < n and (i < lo or (run + cost[i] <= total * r / world + 1e-9 * max(total, 1.0) and i < hi)):
            run += cost[i]
            i += 1
        if i < hi and i < n and run < total * r / world:   # the sample that crosses the mark goes to the earlier slice
            run += cost[i]
            i += 1
        i = max(min(i, hi), min(lo, n))
        cuts.append(i)
    cuts.append(n)
    return [slice(cuts[r], cuts[r + 1]) for r in range(world)]


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def spawn_ranks(world: int, fn, args=()):
    """Starts `world` worker processes on this node (torch.multiprocessing, start method spawn) and calls
    fn(rank, *args, world, port) in each; the workers rendezvous on 127.0.0.1:port.  Returns when all have exited and
    raises if one failed.  fn must be importable from the workers (a module-level function)."""
    import torch.multiprocessing as mp
    port = _free_port()
    mp.spawn(fn, args=tuple(args) + (world, port), nprocs=world, join=True)


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
