"""The N > 1 path of the benchmark on CPU: two `gloo` ranks.  Images are independent, so a
rank's share is a batch of its own and the only exchange is the maximum of the timings."""
from __future__ import annotations

import importlib.util
import os
import sys
from pathlib import Path

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = Path(__file__).resolve().parent.parent


def load_bench():
    spec = importlib.util.spec_from_file_location("bench_module", ROOT / "bench.py")
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod


def _rank_main(rank: int, world: int, port: int, results):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank),
                      WORLD_SIZE=str(world))
    sys.path.insert(0, str(ROOT))
    bench = load_bench()
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        images, dtype, desc = bench.make_workload("mixed", 6, rank)
        digest = sum(int(im.sum()) for im in images)
        shapes = [im.shape for im in images]
        # every rank times its own work; the job's time is the slowest rank's
        mine = [10.0 + rank, 5.0 - rank]
        got = bench.max_over_ranks(mine, dist, torch.device("cpu"))
        results.put((rank, digest, shapes, got, desc, dtype))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_ranks_draw_their_own_batches_and_agree_on_the_slowest_time():
    world = 2
    port = 29500 + (os.getpid() % 2000)
    ctx = mp.get_context("spawn")
    results = ctx.Queue()
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, results)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted(results.get(timeout=240) for _ in range(world))
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    (r0, d0, s0, t0, desc0, dt0), (r1, d1, s1, t1, desc1, dt1) = got
    assert (r0, r1) == (0, 1)
    assert t0 == t1 == [11.0, 5.0]          # element-wise maximum over the ranks
    assert d0 != d1 or s0 != s1             # different ranks, different images
    assert desc0 == desc1 and dt0 == dt1    # same workload description everywhere


def test_a_rank_batch_is_reproducible_and_single_rank_reduction_is_identity():
    bench = load_bench()
    a, _, _ = bench.make_workload("mixed", 5, 1)
    b, _, _ = bench.make_workload("mixed", 5, 1)
    assert all(np.array_equal(x, y) for x, y in zip(a, b))
    assert bench.max_over_ranks([3.0, 4.5], None, None) == [3.0, 4.5]
    cfg = bench.config_of("w", "f16", 256, 4)
    assert cfg["parallelism"].startswith("dp4") and cfg["images_per_step_per_gpu"] == 256
