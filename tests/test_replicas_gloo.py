"""The N > 1 measurement path on CPU: two gloo ranks, barrier + slowest-rank time + aggregation,
and the request-level sharding of a segment table across replicas."""
import os

import numpy as np
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2607_28848_b200 import replicas, synth


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        replicas.barrier()
        ms = 10.0 if rank == 0 else 25.0                     # rank 1 is the slow one
        agg = replicas.aggregate_throughput(units_per_rank_per_step=4096, steps=5, ms_this_rank=ms)
        q.put((rank, agg, replicas.max_over_ranks(rank + 1.5)))
        replicas.barrier()
    finally:
        dist.destroy_process_group()


def test_two_ranks_report_slowest_time_and_summed_work():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = [q.get(timeout=120) for _ in procs]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for _rank, agg, mx in got:
        assert agg["n_gpus"] == 2
        assert abs(agg["ms_per_step"] - 5.0) < 1e-9          # 25 ms / 5 steps: the slowest rank
        assert abs(agg["value"] - 2 * 4096 * 5 / 0.025) < 1e-6
        assert mx == 2.5


def test_single_process_is_the_identity():
    agg = replicas.aggregate_throughput(100, 4, 8.0)
    assert agg == {"n_gpus": 1, "ms_per_step": 2.0, "value": 100 * 4 / 0.008}


def test_shard_segments_keeps_requests_whole_and_balanced():
    segs, rows = synth.cfg3_segments(0)
    shards = replicas.shard_segments(segs.tolist(), 4)
    sizes = [sum(s[1] for s in sh) for sh in shards]
    assert sum(sizes) == rows and max(sizes) - min(sizes) <= 512
    flat = sorted((s[1], s[2], s[3]) for sh in shards for s in sh)
    assert flat == sorted((int(s[1]), int(s[2]), int(s[3])) for s in segs.tolist())
    for sh in shards:                                        # rows renumbered densely from 0
        row = 0
        for st, ln, _ad, _ft in sh:
            assert st == row
            row += ln
