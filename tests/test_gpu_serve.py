"""The batching queue feeding the kernel: requests arriving by a Poisson process (paper Sec. 5
"Input query modeling") wait in the queue of Sec. 2.3 item 2 / Sec. 4.3, and every released batch
goes through preba_preprocess_images on the GPU.  In virtual time the batches must be the batching
oracle's; in real time (preba_serve_run) they must obey the rule's invariants; in both every
request's result must be the transform oracle's."""
from __future__ import annotations

import numpy as np
import pytest

import oracle
from oracle import batching as ob
from paper_2411_19114_b200 import binding as pb
from paper_2411_19114_b200 import workloads as wl

from helpers import MEAN, STD, FP32_TOL, host_threads

pytestmark = pytest.mark.gpu

C, S = 224, 256


def pinned_pool(images):
    """Every image in pinned memory on a 4096-byte boundary, as the in-place mode wants."""
    import torch

    page, starts, at = 4096, [], 0
    for im in images:
        starts.append(at)
        at += -(-im.nbytes // page) * page
    arena = torch.empty(at, dtype=torch.uint8).pin_memory()
    views = []
    for im, st in zip(images, starts):
        v = arena[st:st + im.nbytes].view(im.shape)
        v.copy_(torch.from_numpy(im))
        views.append(v)
    return arena, views


def poisson_arrivals(rate_per_s: float, n: int, seed: int) -> np.ndarray:
    rng = np.random.default_rng(seed)
    gaps = rng.exponential(1e9 / rate_per_s, size=n)
    return np.cumsum(gaps).astype(np.uint64)


def server_staging(batch_max, dev, with_out_host=True):
    import torch

    st = dict(table_host=torch.zeros(16 * batch_max, dtype=torch.uint8).pin_memory(),
              dev_table=torch.empty(16 * batch_max, dtype=torch.uint8, device=dev),
              dev_out=torch.empty((batch_max, 3, C, C), dtype=torch.float32, device=dev),
              dev_status=torch.zeros(1, dtype=torch.int32, device=dev),
              dev_scratch=torch.zeros(pb.SCRATCH_BYTES // 4, dtype=torch.int32, device=dev),
              stream=torch.cuda.Stream(device=dev))
    if with_out_host:
        st["out_host"] = torch.empty((batch_max, 3, C, C), dtype=torch.float32).pin_memory()
    return st


def test_queue_in_virtual_time_feeds_the_kernel_with_the_oracles_batches():
    import torch

    dev = torch.device("cuda:0")
    pool_np = wl.mixed_smooth(24, seed=77)
    _, pool = pinned_pool(pool_np)
    n, batch_max, time_queue = 150, 8, 40_000
    arrivals = [int(t) for t in poisson_arrivals(150_000.0, n, seed=5)]  # mean gap 6.7 us
    image_of = np.random.default_rng(6).integers(0, len(pool), size=n)
    want_batches = ob.batches(arrivals, batch_max, time_queue)
    # the library's queue, looked at at every arrival and every waiting-time limit
    q = pb.PrebaBatcher(batch_max, time_queue)
    got_batches, i, deadline = [], 0, pb.NEVER
    while i < n or deadline != pb.NEVER:
        if i < n and arrivals[i] <= deadline:
            now = arrivals[i]
            q.push(i, now)
            i += 1
        else:
            now = deadline
        ids, deadline = q.poll(now)
        if ids:
            got_batches.append((now, ids))
    assert got_batches == want_batches
    assert sorted(r for _, ids in got_batches for r in ids) == list(range(n))
    # every batch through the kernel, every request against the transform's oracle
    st = server_staging(batch_max, dev)
    want = oracle.preprocess(pool_np, C, S, MEAN, STD, oracle.OUT_F64, nthreads=host_threads())
    for _, ids in got_batches:
        imgs = [pool[int(image_of[r])] for r in ids]
        k = len(ids)
        call = pb.PreparedImages(imgs, st["table_host"], st["out_host"][:k], None, st["dev_table"],
                                 st["dev_out"], C, S, MEAN, STD, pb.F32, stream=st["stream"],
                                 dev_status=st["dev_status"], dev_scratch=st["dev_scratch"],
                                 in_place=True)
        call()
        st["stream"].synchronize()
        got = st["out_host"][:k].numpy()
        for slot, r in enumerate(ids):
            err = float(np.max(np.abs(got[slot].astype(np.float64) - want[int(image_of[r])])))
            assert err <= FP32_TOL, (r, err)
    assert int(st["dev_status"].item()) == 0


def test_real_time_driver_serves_every_request_once_in_order_with_the_oracles_results():
    import torch

    dev = torch.device("cuda:0")
    pool_np = wl.mixed_smooth(16, seed=78)
    _, pool = pinned_pool(pool_np)
    n, batch_max, time_queue, servers = 400, 16, 300_000, 3
    arrivals = poisson_arrivals(40_000.0, n, seed=9)                      # about 10 ms of traffic
    image_of = np.random.default_rng(10).integers(0, len(pool), size=n).astype(np.uint32)
    staging = [server_staging(batch_max, dev, with_out_host=False) for _ in range(servers)]
    arena = torch.full((n, 3, C, C), float("nan"), dtype=torch.float32).pin_memory()
    rec = pb.preba_serve_run(arrivals, image_of, pool, batch_max, time_queue, staging, C, S, MEAN,
                             STD, pb.F32, out_arena=arena)
    torch.cuda.synchronize()
    assert all(int(s["dev_status"].item()) == 0 for s in staging)
    # the batches are consecutive runs that cover every request exactly once
    first, size = rec["batch_first"].astype(np.int64), rec["batch_size"].astype(np.int64)
    assert first[0] == 0 and np.all(first[1:] == first[:-1] + size[:-1]) and first[-1] + size[-1] == n
    assert np.all(size >= 1) and np.all(size <= batch_max)
    assert np.all(rec["batch_server"] < servers)
    done, release = rec["done_ns"], rec["batch_release_ns"]
    for f, k, rel in zip(first, size, release):
        # nobody leaves before arriving; a short batch left because its oldest request had
        # waited Time_queue; a request is done after its batch was released
        assert rel >= arrivals[f + k - 1]
        if k < batch_max:
            assert rel >= arrivals[f] + time_queue
        assert np.all(done[f:f + k] >= rel)
    # every request's result is the oracle's for the image it carried
    want = oracle.preprocess(pool_np, C, S, MEAN, STD, oracle.OUT_F64, nthreads=host_threads())
    got = arena.numpy()
    worst = max(float(np.max(np.abs(got[r].astype(np.float64) - want[int(image_of[r])])))
                for r in range(n))
    assert worst <= FP32_TOL, worst


def test_driver_refuses_bad_arguments_without_starting():
    import ctypes

    sv = pb.PrebaServe()
    nb = ctypes.c_uint32()
    assert pb.lib().preba_serve_run(None, ctypes.byref(nb)) == pb.ERR_INVALID_ARG
    assert pb.lib().preba_serve_run(ctypes.byref(sv), ctypes.byref(nb)) == pb.ERR_INVALID_ARG
