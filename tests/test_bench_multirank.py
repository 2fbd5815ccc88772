"""Host logic of the N > 1 benchmark path on CPU: two gloo ranks, replicas only (no data-path collective).

The path shards by stream: every rank runs its own stream and the only exchange is the max-over-ranks of the
timings, from which rank 0 forms the whole-job figure.  Checked here without a GPU: different ranks get different
streams, the slowest rank decides, and the aggregate counts every rank's units."""
import os
import sys

import numpy as np
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank_main(rank, world, port, q):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    import bench
    from paper_2510_09608_b200 import streamgen as sg
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        wl = sg.workloads()[2]
        stream = sg.Stream(wl, rank)                       # one independent stream per rank
        gids, types, pos = stream.next_chunk()
        first_k = stream.k(0, gids[:1])
        my_ms = 10.0 + 5.0 * rank                          # rank 1 is the slow one
        slowest = bench.max_over_ranks(my_ms, world, device="cpu")
        value = bench.whole_job_value(world, wl.frames, slowest)
        q.put((rank, int(len(gids)), first_k.tobytes(), slowest, value))
    finally:
        dist.destroy_process_group()


def test_two_ranks_replicas_max_timing_and_aggregate():
    world, port = 2, 29571 + os.getpid() % 500
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (_, _, k0, slow0, v0), (_, _, k1, slow1, v1) = res
    assert k0 != k1, "ranks must run different streams"
    assert slow0 == slow1 == 15.0, "the slowest rank's time is what every rank reports"
    assert np.isclose(v0, 2 * 2 / 15e-3) and v0 == v1          # 2 ranks x 2 frames per 15 ms


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, 1) == 3.5
    assert np.isclose(bench.whole_job_value(1, 2, 8.0), 250.0)
