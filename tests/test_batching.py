"""The batching front-end (host only): pins of the plain rule, then the library's queue
against it on seeded Poisson arrivals."""
from __future__ import annotations

import numpy as np
import pytest

from oracle import batching as rule
from paper_2411_19114_b200 import binding as pb
from paper_2411_19114_b200 import build as pbuild


@pytest.fixture(scope="module", autouse=True)
def built_library():
    pbuild.build()


# ---- the rule itself, against cases that can be worked out by hand ------------------------------

def test_rule_full_batches_when_requests_pour_in():
    # 10 requests 1 ns apart, Batch_max 4, long waiting time: 4 + 4 released when the 4th and
    # 8th arrive, the last 2 when request 8 has waited its time
    arr = list(range(100, 110))
    got = rule.batches(arr, 4, 1000)
    assert got == [(103, [0, 1, 2, 3]), (107, [4, 5, 6, 7]), (108 + 1000, [8, 9])]


def test_rule_sparse_requests_leave_alone_after_the_waiting_time():
    arr = [0, 10_000, 20_000]
    assert rule.batches(arr, 8, 500) == [(500, [0]), (10_500, [1]), (20_500, [2])]


def test_rule_a_request_arriving_at_the_limit_still_joins():
    assert rule.batches([0, 500], 8, 500) == [(500, [0, 1])]
    assert rule.batches([0, 501], 8, 500) == [(500, [0]), (1001, [1])]


def test_rule_invariants_on_random_arrivals():
    rng = np.random.default_rng(5)
    for _ in range(50):
        n = int(rng.integers(1, 200))
        arr = np.cumsum(rng.exponential(float(rng.uniform(5, 500)), size=n)).astype(np.int64).tolist()
        bm, tq = int(rng.integers(1, 17)), int(rng.integers(0, 2000))
        got = rule.batches(arr, bm, tq)
        flat = [i for _, ids in got for i in ids]
        assert flat == list(range(n))                       # everyone leaves once, in order
        for t, ids in got:
            assert 1 <= len(ids) <= bm
            assert t >= arr[ids[-1]]                        # nobody leaves before arriving
            assert t - arr[ids[0]] <= tq                    # nobody waits longer than Time_queue
            assert len(ids) == bm or t == arr[ids[0]] + tq  # a short batch leaves at the limit
        assert [t for t, _ in got] == sorted(t for t, _ in got)


def test_params_follow_the_profile():
    # Batch_max = Batch_knee; Time_queue = Time_knee / servers (one big GPU: Time_knee itself)
    assert rule.params(16, 35_000_000, 7) == (16, 5_000_000)
    assert rule.params(128, 35_000_000, 1) == (128, 35_000_000)
    assert pb.preba_batching_params(16, 35_000_000, 7) == (16, 5_000_000)
    assert pb.preba_batching_params(128, 35_000_000, 1) == (128, 35_000_000)
    with pytest.raises(pb.PrebaError):
        pb.preba_batching_params(0, 1, 1)
    with pytest.raises(pb.PrebaError):
        pb.preba_batching_params(1, 1, 0)


# ---- the library's queue against the rule ------------------------------------------------------------

def drive(arr, bm, tq):
    """Feed the queue in virtual time, looking at it at every arrival and every deadline."""
    q = pb.PrebaBatcher(bm, tq)
    got = []
    i, n = 0, len(arr)
    deadline = pb.NEVER
    while i < n or deadline != pb.NEVER:
        if i < n and arr[i] <= deadline:
            now = arr[i]
            while i < n and arr[i] == now:   # everything that arrives now joins before the look
                q.push(i, now)
                i += 1
        else:
            now = deadline
        while True:
            ids, deadline = q.poll(now)
            if not ids:
                break
            got.append((now, ids))
    q.close()
    return got


@pytest.mark.parametrize("seed", range(6))
def test_queue_matches_the_rule_on_poisson_arrivals(seed):
    rng = np.random.default_rng(900 + seed)
    n = int(rng.integers(50, 400))
    mean_gap = float(rng.choice([20, 200, 2000]))
    arr = np.cumsum(rng.exponential(mean_gap, size=n)).astype(np.int64).tolist()
    bm, tq = int(rng.choice([1, 2, 8, 16, 128])), int(rng.choice([0, 300, 1500, 10_000]))
    assert drive(arr, bm, tq) == rule.batches(arr, bm, tq)


def test_queue_rejects_misuse():
    q = pb.PrebaBatcher(4, 100)
    q.push(1, 50)
    with pytest.raises(pb.PrebaError):
        q.push(2, 49)                                     # time runs backwards
    import ctypes
    ids = (ctypes.c_uint64 * 2)()
    assert pb.lib().preba_batcher_poll(q._h, 0, ids, 2, None) == pb.ERR_BUFFER_TOO_SMALL
    assert pb.lib().preba_batcher_poll(None, 0, ids, 4, None) == pb.ERR_INVALID_ARG
    assert q.poll(149) == ([], 150)
    assert q.poll(150) == ([1], pb.NEVER)
    q.close()
    assert pb.lib().preba_batcher_create(0, 5) is None
