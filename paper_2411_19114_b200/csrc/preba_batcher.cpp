// Batching front-end: requests wait in arrival order and leave as a batch when Batch_max are
// queued or the oldest has waited Time_queue (paper Sec. 2.3 item 2, Sec. 4.3).  Host only.
#include <cstdint>
#include <deque>
#include <limits>
#include <mutex>
#include <new>

#include "preba.h"

struct preba_batcher {
  struct Request {
    uint64_t id;
    uint64_t arrival_ns;
  };
  uint32_t batch_max;
  uint64_t time_queue_ns;
  std::mutex lock;
  std::deque<Request> queue;
};

extern "C" int preba_batching_params(uint32_t batch_knee, uint64_t time_knee_ns,
                                     uint32_t n_servers, uint32_t* batch_max,
                                     uint64_t* time_queue_ns) {
  if (batch_knee == 0 || n_servers == 0 || !batch_max || !time_queue_ns)
    return PREBA_ERR_INVALID_ARG;
  *batch_max = batch_knee;                      // Batch_max := Batch_knee
  *time_queue_ns = time_knee_ns / n_servers;    // Time_queue := Time_knee / #servers
  return PREBA_OK;
}

extern "C" preba_batcher_t* preba_batcher_create(uint32_t batch_max, uint64_t time_queue_ns) {
  if (batch_max == 0) return nullptr;
  preba_batcher* b = new (std::nothrow) preba_batcher;
  if (!b) return nullptr;
  b->batch_max = batch_max;
  b->time_queue_ns = time_queue_ns;
  return b;
}

extern "C" void preba_batcher_destroy(preba_batcher_t* b) { delete b; }

extern "C" int preba_batcher_push(preba_batcher_t* b, uint64_t id, uint64_t arrival_ns) {
  if (!b) return PREBA_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> guard(b->lock);
  if (!b->queue.empty() && arrival_ns < b->queue.back().arrival_ns) return PREBA_ERR_INVALID_ARG;
  b->queue.push_back({id, arrival_ns});
  return PREBA_OK;
}

extern "C" int preba_batcher_poll(preba_batcher_t* b, uint64_t now_ns, uint64_t* ids,
                                  uint32_t capacity, uint64_t* next_deadline_ns) {
  if (!b || !ids) return PREBA_ERR_INVALID_ARG;
  if (capacity < b->batch_max) return PREBA_ERR_BUFFER_TOO_SMALL;
  std::lock_guard<std::mutex> guard(b->lock);
  uint32_t take = 0;
  if (b->queue.size() >= b->batch_max) {
    take = b->batch_max;
  } else if (!b->queue.empty()) {
    const uint64_t oldest = b->queue.front().arrival_ns;
    const uint64_t limit = std::numeric_limits<uint64_t>::max() - oldest;
    const uint64_t deadline = b->time_queue_ns > limit ? std::numeric_limits<uint64_t>::max()
                                                        : oldest + b->time_queue_ns;
    if (now_ns >= deadline) take = static_cast<uint32_t>(b->queue.size());
  }
  for (uint32_t i = 0; i < take; ++i) {
    ids[i] = b->queue.front().id;
    b->queue.pop_front();
  }
  if (next_deadline_ns) {
    if (b->queue.empty()) {
      *next_deadline_ns = std::numeric_limits<uint64_t>::max();
    } else {
      const uint64_t oldest = b->queue.front().arrival_ns;
      const uint64_t limit = std::numeric_limits<uint64_t>::max() - oldest;
      *next_deadline_ns = b->time_queue_ns > limit ? std::numeric_limits<uint64_t>::max()
                                                    : oldest + b->time_queue_ns;
    }
  }
  return static_cast<int>(take);
}

// ---- variable-length inputs: one queue per length bucket (paper Sec. 4.3) -------------------------
//
// Requests are sorted into buckets by input length (bucket i holds lengths in
// [i * window, (i + 1) * window); the last bucket also takes everything longer) and every
// bucket has a queue and a Batch_max of its own.  A bucket's batch leaves when Batch_max of
// its requests are queued, or when its oldest request has waited Time_queue; in the second
// case the short batch is filled up from the two adjacent buckets, shorter inputs first,
// never beyond the Batch_max of the longest input in the batch.
#include <vector>

struct preba_bucket_batcher {
  struct Request {
    uint64_t id;
    uint64_t arrival_ns;
  };
  uint64_t window;
  uint64_t time_queue_ns;
  uint64_t last_arrival_ns = 0;
  uint32_t largest_batch = 0;
  std::vector<uint32_t> batch_max;
  std::vector<std::deque<Request>> queue;
  std::mutex lock;

  uint64_t deadline(uint32_t b) const {
    const uint64_t oldest = queue[b].front().arrival_ns;
    const uint64_t limit = std::numeric_limits<uint64_t>::max() - oldest;
    return time_queue_ns > limit ? std::numeric_limits<uint64_t>::max() : oldest + time_queue_ns;
  }
};

extern "C" preba_bucket_batcher_t* preba_bucket_batcher_create(uint32_t n_buckets,
                                                               uint64_t window,
                                                               const uint32_t* batch_max,
                                                               uint64_t time_queue_ns) {
  if (n_buckets == 0 || window == 0 || !batch_max) return nullptr;
  for (uint32_t i = 0; i < n_buckets; ++i)
    if (batch_max[i] == 0) return nullptr;
  preba_bucket_batcher* b = new (std::nothrow) preba_bucket_batcher;
  if (!b) return nullptr;
  b->window = window;
  b->time_queue_ns = time_queue_ns;
  b->batch_max.assign(batch_max, batch_max + n_buckets);
  b->queue.resize(n_buckets);
  for (uint32_t i = 0; i < n_buckets; ++i)
    b->largest_batch = batch_max[i] > b->largest_batch ? batch_max[i] : b->largest_batch;
  return b;
}

extern "C" void preba_bucket_batcher_destroy(preba_bucket_batcher_t* b) { delete b; }

extern "C" int preba_bucket_batcher_push(preba_bucket_batcher_t* b, uint64_t id,
                                         uint64_t arrival_ns, uint64_t length) {
  if (!b) return PREBA_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> guard(b->lock);
  if (arrival_ns < b->last_arrival_ns) return PREBA_ERR_INVALID_ARG;
  b->last_arrival_ns = arrival_ns;
  const uint64_t n = b->queue.size();
  const uint64_t bucket = length / b->window < n ? length / b->window : n - 1;
  b->queue[bucket].push_back({id, arrival_ns});
  return PREBA_OK;
}

extern "C" int preba_bucket_batcher_poll(preba_bucket_batcher_t* b, uint64_t now_ns,
                                         uint64_t* ids, uint32_t capacity,
                                         uint64_t* next_deadline_ns) {
  if (!b || !ids) return PREBA_ERR_INVALID_ARG;
  if (capacity < b->largest_batch) return PREBA_ERR_BUFFER_TOO_SMALL;
  std::lock_guard<std::mutex> guard(b->lock);
  const uint32_t n = static_cast<uint32_t>(b->queue.size());
  uint32_t take = 0;
  auto move_from = [&](uint32_t bucket, uint32_t limit) {
    while (take < limit && !b->queue[bucket].empty()) {
      ids[take++] = b->queue[bucket].front().id;
      b->queue[bucket].pop_front();
    }
  };
  // a bucket that holds its Batch_max leaves as it is (lowest bucket first)
  for (uint32_t i = 0; i < n && take == 0; ++i)
    if (b->queue[i].size() >= b->batch_max[i]) move_from(i, b->batch_max[i]);
  if (take == 0) {
    // else the bucket whose oldest request ran out of waiting time first
    int due = -1;
    uint64_t due_at = 0;
    for (uint32_t i = 0; i < n; ++i) {
      if (b->queue[i].empty()) continue;
      const uint64_t d = b->deadline(i);
      if (d <= now_ns && (due < 0 || d < due_at)) {
        due = static_cast<int>(i);
        due_at = d;
      }
    }
    if (due >= 0) {
      const uint32_t own = static_cast<uint32_t>(due);
      uint32_t limit = b->batch_max[own];
      move_from(own, limit);
      if (own > 0) move_from(own - 1, limit);  // shorter inputs: the limit stays
      if (own + 1 < n) {                       // longer inputs bring their own, lower limit
        limit = b->batch_max[own + 1] < limit ? b->batch_max[own + 1] : limit;
        move_from(own + 1, limit);
      }
    }
  }
  if (next_deadline_ns) {
    uint64_t next = std::numeric_limits<uint64_t>::max();
    for (uint32_t i = 0; i < n; ++i)
      if (!b->queue[i].empty()) next = b->deadline(i) < next ? b->deadline(i) : next;
    *next_deadline_ns = next;
  }
  return static_cast<int>(take);
}
