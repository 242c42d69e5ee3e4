"""TEST INFRASTRUCTURE ONLY: the batching rule of the serving pipeline, stated plainly.

Paper Sec. 2.3 item 2 and Sec. 4.3: single-input requests wait in arrival order; a batch
leaves when Batch_max requests are queued or when the oldest has waited Time_queue, and the
two hyper-parameters come from a profile as Batch_max = Batch_knee and
Time_queue = Time_knee / number of servers.  This is a slow event-by-event statement of that
rule in virtual time (integers, nanoseconds), used to check the library's queue.
"""
from __future__ import annotations


def params(batch_knee: int, time_knee_ns: int, n_servers: int) -> tuple[int, int]:
    return batch_knee, time_knee_ns // n_servers


def batches(arrivals_ns: list[int], batch_max: int, time_queue_ns: int) -> list[tuple[int, list[int]]]:
    """(release time, request indices) of every batch, for requests 0..n-1 arriving at the
    given non-decreasing times, when the queue is looked at exactly at every arrival and
    every waiting-time limit."""
    out = []
    waiting: list[int] = []          # indices of queued requests, oldest first
    i, n = 0, len(arrivals_ns)
    while i < n or waiting:
        limit = arrivals_ns[waiting[0]] + time_queue_ns if waiting else None
        if i < n and (limit is None or arrivals_ns[i] <= limit):
            # the next thing to happen is an arrival (an arrival at the very limit is still
            # in time to join: the queue is looked at after it has been added)
            now = arrivals_ns[i]
            waiting.append(i)
            i += 1
            if len(waiting) >= batch_max:
                out.append((now, waiting[:batch_max]))
                waiting = waiting[batch_max:]
            elif limit is not None and now >= limit:
                out.append((now, waiting))
                waiting = []
        else:
            out.append((limit, waiting))
            waiting = []
    return out


def bucket_of(length: int, window: int, n_buckets: int) -> int:
    """Sec. 4.3: lengths are bucketised into non-overlapping windows; the last bucket is open."""
    return min(n_buckets - 1, length // window)


def bucketed_batches(arrivals_ns: list[int], lengths: list[int], window: int,
                     batch_max: list[int], time_queue_ns: int) -> list[tuple[int, list[int]]]:
    """(release time, request indices) of every batch of the bucketised system of Sec. 4.3,
    when the queues are looked at exactly at every arrival and every waiting-time limit, one
    batch after the other until none is due.

    A bucket is due when it holds its Batch_max (full buckets first, lowest first; it releases
    its oldest Batch_max), or when its oldest request has waited Time_queue (earliest limit
    first).  A bucket released by the time limit is short: it is filled from the lower
    neighbour, then from the upper neighbour, oldest first, and the batch never exceeds the
    Batch_max of the longest input's bucket."""
    n_b = len(batch_max)
    waiting: list[list[int]] = [[] for _ in range(n_b)]
    out: list[tuple[int, list[int]]] = []

    def release(now: int) -> bool:
        for b in range(n_b):
            if len(waiting[b]) >= batch_max[b]:
                out.append((now, waiting[b][:batch_max[b]]))
                del waiting[b][:batch_max[b]]
                return True
        due = [(arrivals_ns[waiting[b][0]] + time_queue_ns, b) for b in range(n_b) if waiting[b]]
        due = [d for d in due if d[0] <= now]
        if not due:
            return False
        _, b = min(due)
        batch = waiting[b][:]
        waiting[b].clear()
        limit = batch_max[b]
        if b > 0:
            while len(batch) < limit and waiting[b - 1]:
                batch.append(waiting[b - 1].pop(0))
        if b + 1 < n_b:
            limit = min(limit, batch_max[b + 1])
            while len(batch) < limit and waiting[b + 1]:
                batch.append(waiting[b + 1].pop(0))
        out.append((now, batch))
        return True

    i, n = 0, len(arrivals_ns)
    while i < n or any(waiting):
        limits = [arrivals_ns[w[0]] + time_queue_ns for w in waiting if w]
        limit = min(limits) if limits else None
        if i < n and (limit is None or arrivals_ns[i] <= limit):
            now = arrivals_ns[i]
            waiting[bucket_of(lengths[i], window, n_b)].append(i)
            i += 1
        else:
            now = limit
        while release(now):
            pass
    return out
