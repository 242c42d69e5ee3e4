// Serving driver: single-image requests arrive in real time, wait in the batching queue
// (paper Sec. 2.3 item 2, Sec. 4.3) and leave as batches to the servers that share the GPU
// (Sec. 3), each of which runs its batches through preba_preprocess_images on a stream of its
// own.  A measuring aid like preba_preprocess_repeated: it creates threads and waits for
// streams.  One thread feeds the queue at the requests' arrival times (Sec. 5 "Input query
// modeling": the caller draws them, e.g. from a Poisson process); one thread per server polls
// the queue, and a released batch goes to whichever server asks first.
#include <cuda_runtime.h>

#include <atomic>
#include <chrono>
#include <cstdint>
#include <thread>
#include <vector>

#include "preba.h"
#include "preba_internal.h"

namespace {

using Clock = std::chrono::steady_clock;

uint64_t since(const Clock::time_point& start) {
  return static_cast<uint64_t>(
      std::chrono::duration_cast<std::chrono::nanoseconds>(Clock::now() - start).count());
}

inline void relax() {
#if defined(__x86_64__) || defined(__i386__)
  __builtin_ia32_pause();
#else
  std::this_thread::yield();
#endif
}

struct Shared {
  const preba_serve_t* s;
  preba_batcher_t* queue;
  Clock::time_point start;
  std::atomic<uint32_t> served{0};
  std::atomic<uint32_t> batches{0};
  std::atomic<int> error{PREBA_OK};
  std::atomic<int> cuda_error{0};
};

void feed(Shared* sh) {
  const preba_serve_t& s = *sh->s;
  for (uint32_t i = 0; i < s.n_requests; ++i) {
    // a request enters the queue no earlier than its arrival time; its waiting time counts
    // from the arrival time even if this thread is late
    while (since(sh->start) < s.arrival_ns[i]) {
      if (sh->error.load(std::memory_order_relaxed) != PREBA_OK) return;
      relax();
    }
    const int rc = preba_batcher_push(sh->queue, i, s.arrival_ns[i]);
    if (rc != PREBA_OK) {
      sh->error.store(rc);
      return;
    }
  }
}

void serve(Shared* sh, uint32_t server) {
  const preba_serve_t& s = *sh->s;
  if (cudaSetDevice(s.device) != cudaSuccess) {
    sh->error.store(PREBA_ERR_CUDA);
    return;
  }
  std::vector<uint64_t> ids(s.batch_max);
  std::vector<const uint8_t*> images(s.batch_max);
  std::vector<uint32_t> h(s.batch_max), w(s.batch_max);
  const uint64_t per_image = 3ull * s.out_size * s.out_size * preba::dtype_bytes(s.out_dtype);
  cudaStream_t stream = static_cast<cudaStream_t>(s.streams[server]);
  while (sh->served.load(std::memory_order_acquire) < s.n_requests) {
    if (sh->error.load(std::memory_order_relaxed) != PREBA_OK) return;
    const uint64_t now = since(sh->start);
    const int k = preba_batcher_poll(sh->queue, now, ids.data(), s.batch_max, nullptr);
    if (k < 0) {
      sh->error.store(k);
      return;
    }
    if (k == 0) {
      for (int i = 0; i < 64; ++i) relax();
      continue;
    }
    const uint64_t released = since(sh->start);  // the batch is in this server's hands
    for (int i = 0; i < k; ++i) {
      const uint32_t which = s.image_index[ids[i]];
      images[i] = s.pool_images[which];
      h[i] = s.pool_h[which];
      w[i] = s.pool_w[which];
    }
    preba_image_batch_t b = {};
    b.images = images.data();
    b.h = h.data();
    b.w = w.data();
    b.n = static_cast<uint32_t>(k);
    b.flags = PREBA_IMAGES_IN_PLACE;
    b.table_host = s.table_host[server];
    // requests leave in arrival order, so a batch is a run of consecutive requests and its
    // results are a contiguous piece of the arena
    b.out_host = s.out_arena ? static_cast<uint8_t*>(s.out_arena) + ids[0] * per_image
                             : s.out_host[server];
    b.out_bytes = static_cast<uint64_t>(k) * per_image;
    b.dev_table = s.dev_table[server];
    b.dev_out = s.dev_out[server];
    b.dev_status = s.dev_status ? s.dev_status[server] : nullptr;
    b.dev_scratch = s.dev_scratch ? s.dev_scratch[server] : nullptr;
    int rc = preba_preprocess_images(&b, s.out_size, s.resize_short, s.mean, s.std, s.out_dtype,
                                     stream);
    if (rc == PREBA_OK && cudaStreamSynchronize(stream) != cudaSuccess) {
      sh->cuda_error.store(static_cast<int>(cudaGetLastError()));
      rc = PREBA_ERR_CUDA;
    }
    if (rc != PREBA_OK) {
      sh->error.store(rc);
      return;
    }
    const uint64_t done = since(sh->start);
    const uint32_t slot = sh->batches.fetch_add(1);
    s.batch_size[slot] = static_cast<uint32_t>(k);
    s.batch_first[slot] = static_cast<uint32_t>(ids[0]);
    s.batch_release_ns[slot] = released;
    s.batch_server[slot] = server;
    for (int i = 0; i < k; ++i) s.done_ns[ids[i]] = done;
    sh->served.fetch_add(static_cast<uint32_t>(k), std::memory_order_release);
  }
}

}  // namespace

extern "C" int preba_serve_run(const preba_serve_t* s, uint32_t* n_batches) {
  if (!s || !n_batches || !s->arrival_ns || !s->image_index || s->n_requests == 0 ||
      !s->pool_images || !s->pool_h || !s->pool_w || s->pool_size == 0 || s->batch_max == 0 ||
      s->n_servers == 0 || s->n_servers > 64 || !s->table_host || !s->dev_table || !s->dev_out ||
      !s->streams || !s->done_ns || !s->batch_size || !s->batch_first || !s->batch_release_ns ||
      !s->batch_server || (!s->out_arena && !s->out_host) || !preba::dtype_ok(s->out_dtype))
    return PREBA_ERR_INVALID_ARG;
  for (uint32_t i = 0; i < s->n_requests; ++i) {
    if (s->image_index[i] >= s->pool_size) return PREBA_ERR_INVALID_ARG;
    if (i && s->arrival_ns[i] < s->arrival_ns[i - 1]) return PREBA_ERR_INVALID_ARG;
  }
  for (uint32_t v = 0; v < s->n_servers; ++v)
    if (!s->table_host[v] || !s->dev_table[v] || !s->dev_out[v] ||
        (!s->out_arena && !s->out_host[v]))
      return PREBA_ERR_INVALID_ARG;
  Shared sh;
  sh.s = s;
  sh.queue = preba_batcher_create(s->batch_max, s->time_queue_ns);
  if (!sh.queue) return PREBA_ERR_INVALID_ARG;
  sh.start = Clock::now();
  std::vector<std::thread> threads;
  threads.emplace_back(feed, &sh);
  for (uint32_t v = 0; v < s->n_servers; ++v) threads.emplace_back(serve, &sh, v);
  for (auto& t : threads) t.join();
  preba_batcher_destroy(sh.queue);
  *n_batches = sh.batches.load();
  const int rc = sh.error.load();
  if (rc == PREBA_ERR_CUDA) preba::g_last_cuda_error = sh.cuda_error.load();
  return rc;
}
