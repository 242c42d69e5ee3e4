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
