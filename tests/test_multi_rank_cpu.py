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
