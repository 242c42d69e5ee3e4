// Host-side entry points that need no device: sizes, packing, error text.
#include <algorithm>
#include <cstring>
#include <thread>
#include <vector>

#include "preba.h"
#include "preba_internal.h"

namespace preba {

bool dtype_ok(int out_dtype) {
  return out_dtype == PREBA_F32 || out_dtype == PREBA_F16 || out_dtype == PREBA_BF16;
}

uint32_t dtype_bytes(int out_dtype) {
  return out_dtype == PREBA_F32 ? 4u : out_dtype == PREBA_U8 ? 1u : 2u;
}

uint64_t align_up(uint64_t v, uint64_t a) { return (v + a - 1) / a * a; }

bool dims_ok(uint32_t h, uint32_t w) {
  return h >= 1 && w >= 1 && h <= PREBA_MAX_DIM && w <= PREBA_MAX_DIM;
}

}  // namespace preba

extern "C" int preba_query(const uint32_t* h, const uint32_t* w, uint32_t n, uint32_t out_size,
                           int out_dtype, preba_sizes_t* sizes) {
  if (!h || !w || !sizes || n == 0 || out_size == 0 || out_size > PREBA_MAX_RESIZE ||
      !preba::dtype_ok(out_dtype))
    return PREBA_ERR_INVALID_ARG;
  uint64_t at = 0;
  for (uint32_t i = 0; i < n; ++i) {
    if (!preba::dims_ok(h[i], w[i])) return PREBA_ERR_INVALID_ARG;
    at = preba::align_up(at + 3ull * h[i] * w[i], PREBA_PACK_ALIGN);
  }
  sizes->packed_bytes = at;
  sizes->table_bytes = static_cast<uint64_t>(n) * sizeof(preba_img_t);
  sizes->out_bytes = static_cast<uint64_t>(n) * 3ull * out_size * out_size *
                     preba::dtype_bytes(out_dtype);
  sizes->align = PREBA_PACK_ALIGN;
  sizes->reserved = 0;
  return PREBA_OK;
}

extern "C" int preba_pack(const uint8_t* const* images, const uint32_t* h, const uint32_t* w,
                          uint32_t n, uint8_t* packed, uint64_t capacity, preba_img_t* table) {
  if (!images || !h || !w || !packed || !table || n == 0) return PREBA_ERR_INVALID_ARG;
  uint64_t need = 0;
  for (uint32_t i = 0; i < n; ++i) {
    if (!images[i] || !preba::dims_ok(h[i], w[i])) return PREBA_ERR_INVALID_ARG;
    need = preba::align_up(need + 3ull * h[i] * w[i], PREBA_PACK_ALIGN);
  }
  if (capacity < need) return PREBA_ERR_BUFFER_TOO_SMALL;
  uint64_t at = 0;
  for (uint32_t i = 0; i < n; ++i) {
    table[i].offset = at;
    table[i].h = h[i];
    table[i].w = w[i];
    at = preba::align_up(at + 3ull * h[i] * w[i], PREBA_PACK_ALIGN);
  }
  // the copies: images are independent, so large batches are split over a few threads
  // (contiguous runs of images of about equal bytes)
  auto copy_run = [&](uint32_t first, uint32_t last) {
    for (uint32_t i = first; i < last; ++i) {
      const uint64_t bytes = 3ull * h[i] * w[i];
      const uint64_t off = table[i].offset;
      std::memcpy(packed + off, images[i], bytes);
      const uint64_t next = preba::align_up(off + bytes, PREBA_PACK_ALIGN);
      std::memset(packed + off + bytes, 0, next - (off + bytes));
    }
  };
  constexpr uint64_t kBytesPerThread = 4ull << 20;
  const unsigned hw = std::max(1u, std::thread::hardware_concurrency());
  const unsigned workers = static_cast<unsigned>(
      std::min<uint64_t>({8, hw, need / kBytesPerThread, static_cast<uint64_t>(n)}));
  if (workers <= 1) {
    copy_run(0, n);
  } else {
    std::vector<std::thread> pool;
    uint32_t first = 0;
    for (unsigned t = 0; t < workers; ++t) {
      // run t ends where the byte count passes its share
      uint32_t last = first;
      const uint64_t goal = need * (t + 1) / workers;
      while (last < n && (t + 1 == workers || table[last].offset < goal)) ++last;
      if (t + 1 == workers) last = n;
      pool.emplace_back(copy_run, first, last);
      first = last;
    }
    for (auto& th : pool) th.join();
  }
  return PREBA_OK;
}

extern "C" const char* preba_strerror(int code) {
  switch (code) {
    case PREBA_OK: return "ok";
    case PREBA_ERR_INVALID_ARG: return "invalid argument";
    case PREBA_ERR_BUFFER_TOO_SMALL: return "buffer too small";
    case PREBA_ERR_BAD_TABLE: return "bad image table entry";
    case PREBA_ERR_CUDA: return "CUDA runtime error";
    case PREBA_ERR_TIMEOUT: return "device wait ran out";
    case PREBA_ERR_TOO_LARGE: return "batch exceeds the library's built-in staging space, or an image is reduced by more than the kernel can hold";
    case PREBA_ERR_BAD_CROP: return "crop window outside the resized image";
    case PREBA_ERR_UNSUPPORTED: return "a JPEG stream of a kind that is not decoded";
    case PREBA_ERR_BAD_STREAM: return "a malformed or truncated JPEG stream";
    case PREBA_ERR_RANGE: return "an index left its range inside a kernel (checked build)";
    default: return "unknown preba error code";
  }
}
