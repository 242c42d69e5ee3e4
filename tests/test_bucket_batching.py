"""The batching front-end for variable-length inputs (paper Sec. 4.3): pins of the plain
statement of the rule, then the library's queues against it on seeded Poisson arrivals with
utterance-like lengths.  Host only."""
from __future__ import annotations

import ctypes

import numpy as np
import pytest

from oracle import batching as rule
from paper_2411_19114_b200 import binding as pb
from paper_2411_19114_b200 import build as pbuild


@pytest.fixture(scope="module", autouse=True)
def built_library():
    pbuild.build()


W = 2500                                   # bucket window: 2.5 s in milliseconds (the paper's)
BM = [16, 12, 8, 6, 4, 2]                  # Batch_max per bucket: smaller for longer inputs


# ---- the rule, against cases worked out by hand -------------------------------------------------

def test_buckets_are_non_overlapping_windows_with_an_open_last_one():
    assert [rule.bucket_of(x, W, 6) for x in (0, 2499, 2500, 4999, 6000, 12_499, 12_500, 99_000)] \
        == [0, 0, 1, 1, 2, 4, 5, 5]


def test_the_papers_example_four_requests_of_six_seconds_form_one_batch():
    # Fig. "dynamic batching system": a 6 s input falls under the third bucket and is coalesced
    # with the three waiting there into a batch of 4
    arr = [0, 10, 20, 30]
    got = rule.bucketed_batches(arr, [6000, 5500, 7000, 6000], W, [16, 12, 4, 2], 1_000_000)
    assert got == [(30, [0, 1, 2, 3])]


def test_a_full_bucket_leaves_at_once_and_others_keep_waiting():
    arr = [0, 1, 2, 3, 4]
    lens = [100, 3000, 200, 300, 3100]                     # buckets 0 1 0 0 1
    got = rule.bucketed_batches(arr, lens, W, [3, 8], 1000)
    # bucket 0 holds its Batch_max (3) when request 3 arrives; bucket 1's two requests run out
    # of waiting time at 1 + 1000 and find nothing to merge with
    assert got == [(3, [0, 2, 3]), (1001, [1, 4])]


def test_a_short_batch_is_filled_from_the_lower_then_the_upper_neighbour():
    arr = [0, 5, 6, 7, 8, 9]
    lens = [6000, 3000, 3100, 9000, 8000, 100]             # buckets 2 1 1 3 3 0
    bm = [8, 8, 4, 3]
    got = rule.bucketed_batches(arr, lens, W, bm, 100)
    # at 100 request 0 (bucket 2) has waited its time: own [0], lower neighbour (bucket 1)
    # gives 1, 2 (limit 4 stays), the upper neighbour's Batch_max is 3: the batch already
    # holds 3, so none of bucket 3 joins; bucket 0 is not adjacent.  Bucket 3's requests leave
    # at 7 + 100 with nothing left to merge in bucket 2; bucket 0's at 9 + 100.
    assert got == [(100, [0, 1, 2]), (107, [3, 4]), (109, [5])]


def test_merging_from_a_longer_bucket_is_capped_by_that_buckets_batch_max():
    arr = [0, 1, 2, 3]
    lens = [100, 200, 2600, 2700]                          # buckets 0 0 1 1
    got = rule.bucketed_batches(arr, lens, W, [8, 3], 50)
    # bucket 0 is due at 50 with two requests; the upper neighbour caps the batch at its own
    # Batch_max 3, so only one of its two requests joins; the other leaves at 3 + 50
    assert got == [(50, [0, 1, 2]), (53, [3])]
    got = rule.bucketed_batches(arr, lens, W, [8, 4], 50)
    assert got == [(50, [0, 1, 2, 3])]                     # cap 4: both join
    got = rule.bucketed_batches(arr, lens, W, [8, 1], 50)
    # bucket 1 (Batch_max 1) releases each of its requests as it arrives; bucket 0 alone at 50
    assert got == [(2, [2]), (3, [3]), (50, [0, 1])]


def test_buckets_due_at_the_same_time_go_lowest_first():
    # both requests run out of waiting time at 50: bucket 0 goes first and takes its upper
    # neighbour's request along
    assert rule.bucketed_batches([0, 0], [100, 2600], W, [8, 8], 50) == [(50, [0, 1])]
    # three buckets due together, no merging possible beyond neighbours' contents
    got = rule.bucketed_batches([0, 0, 0], [100, 2600, 9000], W, [8, 8, 8, 8], 50)
    assert got == [(50, [0, 1]), (50, [2])]


def test_one_bucket_is_the_plain_rule():
    rng = np.random.default_rng(1)
    for _ in range(20):
        n = int(rng.integers(1, 150))
        arr = np.cumsum(rng.exponential(float(rng.uniform(5, 500)), size=n)).astype(np.int64).tolist()
        lens = rng.integers(0, 40_000, size=n).tolist()
        bm, tq = int(rng.integers(1, 17)), int(rng.integers(0, 2000))
        assert rule.bucketed_batches(arr, lens, W, [bm], tq) == rule.batches(arr, bm, tq)


def lengths_like_read_speech(rng, n):
    """Utterance lengths in ms: most between 2 and 17 s, a tail up to 35 s."""
    return np.clip(rng.gamma(4.0, 3000.0, size=n), 1000, 35_000).astype(np.int64).tolist()


def test_rule_invariants_on_random_traffic():
    rng = np.random.default_rng(2)
    for _ in range(40):
        n = int(rng.integers(1, 300))
        arr = np.cumsum(rng.exponential(float(rng.uniform(5, 800)), size=n)).astype(np.int64).tolist()
        lens = lengths_like_read_speech(rng, n)
        tq = int(rng.integers(0, 3000))
        got = rule.bucketed_batches(arr, lens, W, BM, tq)
        flat = sorted(i for _, ids in got for i in ids)
        assert flat == list(range(n))                                   # everyone leaves exactly once
        assert [t for t, _ in got] == sorted(t for t, _ in got)
        for t, ids in got:
            buckets = [rule.bucket_of(lens[i], W, len(BM)) for i in ids]
            assert len(ids) <= BM[max(buckets)]                         # the longest input's limit
            assert max(buckets) - min(buckets) <= 2                     # own bucket and its neighbours
            own = buckets[0]
            assert all(abs(b - own) <= 1 for b in buckets)
            assert all(t >= arr[i] for i in ids)                        # nobody leaves before arriving
            assert all(t - arr[i] <= tq for i in ids)                   # nobody waits beyond Time_queue
            for b in set(buckets):                                      # first come, first served per bucket
                mine = [i for i, bb in zip(ids, buckets) if bb == b]
                assert mine == sorted(mine)


# ---- the library's queues against the rule --------------------------------------------------------

def drive(arr, lens, window, bm, tq):
    q = pb.BucketBatcher(window, bm, tq)
    got = []
    i, n = 0, len(arr)
    deadline = pb.NEVER
    while i < n or deadline != pb.NEVER:
        if i < n and arr[i] <= deadline:
            now = arr[i]
            q.push(i, now, lens[i])        # one request per look, as the rule states it
            i += 1
        else:
            now = deadline
        while True:
            ids, deadline = q.poll(now)
            if not ids:
                break
            got.append((now, ids))
    return got


@pytest.mark.parametrize("seed", range(8))
def test_queues_match_the_rule_on_poisson_arrivals(seed):
    rng = np.random.default_rng(700 + seed)
    n = int(rng.integers(50, 500))
    arr = np.cumsum(rng.exponential(float(rng.choice([20, 200, 2000])), size=n)).astype(np.int64).tolist()
    lens = lengths_like_read_speech(rng, n)
    bm = [BM, [4, 4, 4, 4], [1, 2, 3], [32, 1, 32, 1, 32]][seed % 4]
    tq = int(rng.choice([0, 300, 1500, 10_000]))
    assert drive(arr, lens, W, bm, tq) == rule.bucketed_batches(arr, lens, W, bm, tq)


def test_hand_worked_cases_through_the_library():
    assert drive([0, 5, 6, 7, 8, 9], [6000, 3000, 3100, 9000, 8000, 100], W, [8, 8, 4, 3], 100) \
        == [(100, [0, 1, 2]), (107, [3, 4]), (109, [5])]
    assert drive([0, 10, 20, 30], [6000, 5500, 7000, 6000], W, [16, 12, 4, 2], 1_000_000) \
        == [(30, [0, 1, 2, 3])]


def test_queues_reject_misuse():
    L = pb.lib()
    bm = (ctypes.c_uint32 * 2)(4, 2)
    assert L.preba_bucket_batcher_create(0, 10, bm, 5) is None
    assert L.preba_bucket_batcher_create(2, 0, bm, 5) is None
    assert L.preba_bucket_batcher_create(2, 10, None, 5) is None
    zero = (ctypes.c_uint32 * 2)(4, 0)
    assert L.preba_bucket_batcher_create(2, 10, zero, 5) is None
    q = pb.BucketBatcher(10, [4, 2], 100)
    q.push(1, 50, 3)
    with pytest.raises(pb.PrebaError):
        q.push(2, 49, 3)                                   # time runs backwards
    ids = (ctypes.c_uint64 * 3)()
    assert L.preba_bucket_batcher_poll(q._h, 0, ids, 3, None) == pb.ERR_BUFFER_TOO_SMALL
    assert L.preba_bucket_batcher_poll(None, 0, ids, 4, None) == pb.ERR_INVALID_ARG
    assert q.poll(149) == ([], 150)
    assert q.poll(150) == ([1], pb.NEVER)
