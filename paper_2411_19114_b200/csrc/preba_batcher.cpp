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
