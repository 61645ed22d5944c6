"""The multi-GPU path's host logic on two CPU ranks (gloo): sample sharding, per-rank seeds, and the whole-job
throughput = units of all ranks / time of the slowest rank."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        import workloads as wk
        from paper_2505_01068_b200 import shard

        wl = wk.WORKLOADS[3]
        # strong scaling: each rank takes its slice of one common batch
        sl = shard.batch_slice(wl.batch + 1, world, rank)
        # weak scaling: each rank draws its own batch
        valid = wk.draw_valid_len(np.random.default_rng(shard.rank_seed(wl.seed, rank)), wl)
        tokens = int(valid.sum())
        ms = 2.0 + rank  # rank 1 is the slow one
        total, t_max, per_s = shard.job_throughput(tokens, ms)
        gathered = [None] * world
        dist.all_gather_object(gathered, (sl.start, sl.stop, tokens, valid[:2].tolist()))
        out[rank] = (total, t_max, per_s, gathered)
    finally:
        dist.destroy_process_group()


def test_two_rank_sharding_and_job_throughput():
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert set(res) == {0, 1}
    total0, tmax0, per_s0, gathered = res[0]
    assert res[1][:3] == (total0, tmax0, per_s0)                # every rank computes the same job figures
    (a0, b0, tok0, v0), (a1, b1, tok1, v1) = gathered
    assert a0 == 0 and b0 == a1 and b1 == 33 and abs((b0 - a0) - (b1 - a1)) <= 1   # slices tile the batch, balanced
    assert v0 != v1                                              # independent per-rank draws
    assert total0 == tok0 + tok1 and tmax0 == 3.0
    assert abs(per_s0 - (tok0 + tok1) / 3.0e-3) < 1e-6 * per_s0


def test_single_process_and_slices_cover_every_batch():
    from paper_2505_01068_b200 import shard

    assert shard.job_throughput(1000, 4.0) == (1000.0, 4.0, 250000.0)
    for batch in (0, 1, 7, 64, 65):
        for world in (1, 2, 3, 8):
            idx = [i for r in range(world) for i in range(batch)[shard.batch_slice(batch, world, r)]]
            assert idx == list(range(batch))


def test_stack_chunks_tile_the_batch():
    """Host logic of the stack's concurrent issue: the groups of samples cover the batch once, in order, balanced, and
    collapse to one group when everything is issued on the caller's stream."""
    from paper_2505_01068_b200.stack import GsitStack

    layer = [{}]
    for batch in (1, 2, 5, 64):
        for chunks in (1, 2, 3, 8):
            st = GsitStack(layer, layer, layer, (4, 4, 4), 2, 2, batch_chunks=chunks)
            sl = st._chunks(batch)
            assert len(sl) == min(chunks, batch)
            assert sl[0].start == 0 and sl[-1].stop == batch
            assert all(a.stop == b.start for a, b in zip(sl, sl[1:]))
            sizes = [s.stop - s.start for s in sl]
            assert max(sizes) - min(sizes) <= 1 and min(sizes) >= 1
            st.concurrent_rings = False
            assert st._chunks(batch) == [slice(0, batch)]


def _stub_rank(rank, tag, out, world, port):
    """What bench.py's workers do around the step, with a stub step and gloo instead of NCCL."""
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from paper_2505_01068_b200 import shard
        dist.barrier()
        total, t_max, per_s = shard.job_throughput(100 * (rank + 1), 1.0 + rank)
        out[rank] = (tag, world, total, t_max)
    finally:
        dist.destroy_process_group()


def test_spawn_ranks_starts_one_worker_per_rank_and_they_rendezvous():
    """The launcher bench.py uses for --gpus N without torchrun: N workers, ranks 0..N-1, one rendezvous, job figures equal."""
    from paper_2505_01068_b200 import shard

    with mp.Manager() as mgr:
        out = mgr.dict()
        shard.spawn_ranks(2, _stub_rank, ("tag", out))
        res = dict(out)
    assert res == {0: ("tag", 2, 300.0, 2.0), 1: ("tag", 2, 300.0, 2.0)}


def test_bench_selects_the_launcher_only_without_a_torchrun_environment(monkeypatch):
    """`python bench.py --gpus 2` spawns its ranks; under torchrun (WORLD_SIZE set) the process is one of the ranks."""
    import importlib.util
    import sys
    from pathlib import Path
    from paper_2505_01068_b200 import shard

    spec = importlib.util.spec_from_file_location("bench_under_test", Path(__file__).resolve().parent.parent / "bench.py")
    bench = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(bench)
    calls = []
    monkeypatch.setattr(shard, "spawn_ranks", lambda world, fn, args=(): calls.append(("spawn", world, fn.__name__)))
    monkeypatch.setattr(bench, "run_gpu", lambda args: calls.append(("run", args.gpus)))
    monkeypatch.delenv("WORLD_SIZE", raising=False)
    monkeypatch.setattr(sys, "argv", ["bench.py", "--gpus", "2", "--steps", "3"])
    bench.main()
    monkeypatch.setenv("WORLD_SIZE", "2")
    bench.main()
    monkeypatch.delenv("WORLD_SIZE")
    monkeypatch.setattr(sys, "argv", ["bench.py", "--steps", "3"])
    bench.main()
    assert calls == [("spawn", 2, "_spawned_rank"), ("run", 2), ("run", 1)]


def test_balanced_slices_follow_the_valid_tokens():
    import workloads as wk
    from paper_2505_01068_b200 import shard

    wl = wk.WORKLOADS[4]
    valid = wk.draw_valid_len(np.random.default_rng(wl.seed), wl)
    cost = valid.sum(axis=1)
    for world in (1, 2, 3, 8):
        sl = shard.balanced_slices(cost, world)
        assert [i for s in sl for i in range(wl.batch)[s]] == list(range(wl.batch))
        shares = [int(cost[s].sum()) for s in sl]
        assert max(shares) - min(shares) <= 2 * int(cost.max()) and min(shares) > 0
    # a heavy sample at one end moves the cut, unlike a split by count
    assert shard.balanced_slices([1000, 1, 1, 1], 2) == [slice(0, 1), slice(1, 4)]
    assert shard.balanced_slices([1, 1, 1, 1000], 2) == [slice(0, 3), slice(3, 4)]
    for n, world in ((0, 2), (1, 3), (2, 2), (5, 8)):
        sl = shard.balanced_slices([7] * n, world)
        assert len(sl) == world and [i for s in sl for i in range(n)[s]] == list(range(n))
