// Fused resize -> center crop -> normalise -> HWC->NCHW for a ragged batch (sm_100a).
//
// One launch per batch.  A CTA owns a slab of output rows of one image, reads
// the image's {offset, h, w} from the device table, derives the sampling grid
// in exact integers, interpolates in fp32 and stores planar output.
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <cmath>

#include "preba.h"
#include "preba_internal.h"

namespace preba {

constexpr int kThreads = 256;
constexpr uint32_t kSlabRows = 8;

struct Params {
  const uint8_t* pixels;
  uint64_t pixels_bytes;
  const preba_img_t* table;
  void* out;
  int32_t* status;
  uint32_t n;
  uint32_t C;      // crop side
  uint32_t S;      // resized shorter side
  uint32_t slabs;  // slabs per image
  float a[3];      // 1 / (255 * std_c)
  float b[3];      // -mean_c / std_c
};

// Taps and weight of one crop-window index along one axis: the source
// coordinate ((origin + j) + 1/2) * in / r - 1/2, clamped to [0, in - 1], as
// num / den with num = (2X + 1) * in - r and den = 2r.
struct Tap {
  uint32_t i0;
  uint32_t i1;
  float lam;
};

__device__ __forceinline__ Tap axis_tap(uint32_t in, uint64_t r, uint64_t origin, uint32_t j) {
  const uint64_t X = origin + j;
  const uint64_t den = 2 * r;
  const uint64_t pos = (2 * X + 1) * in;  // < 2^46
  uint64_t num = pos > r ? pos - r : 0;
  const uint64_t hi = static_cast<uint64_t>(in - 1) * den;
  num = num < hi ? num : hi;
  uint64_t q, rem;
  if ((num | den) >> 32) {
    q = num / den;
    rem = num - q * den;
  } else {
    const uint32_t n32 = static_cast<uint32_t>(num), d32 = static_cast<uint32_t>(den);
    const uint32_t q32 = n32 / d32;
    q = q32;
    rem = n32 - q32 * d32;
  }
  Tap t;
  t.i0 = static_cast<uint32_t>(q);
  t.i1 = t.i0 + 1 < in ? t.i0 + 1 : in - 1;
  t.lam = static_cast<float>(rem) / static_cast<float>(den);
  return t;
}

__device__ __forceinline__ void report(int32_t* status, int code) {
  if (status) atomicCAS(status, 0, code);
}

__device__ __forceinline__ bool entry_ok(const preba_img_t& e, uint64_t pixels_bytes) {
  if (e.h == 0 || e.w == 0 || e.h > PREBA_MAX_DIM || e.w > PREBA_MAX_DIM) return false;
  if (e.offset % PREBA_PACK_ALIGN) return false;
  const uint64_t bytes = 3ull * e.h * e.w;
  return e.offset <= pixels_bytes && bytes <= pixels_bytes - e.offset;
}

__device__ __forceinline__ void store_out(float* p, float v) { *p = v; }
__device__ __forceinline__ void store_out(__half* p, float v) { *p = __float2half_rn(v); }

// Direct path: every tap is fetched from global memory.  Serves any image size.
template <typename OutT>
__global__ void __launch_bounds__(kThreads) preba_gather_kernel(const Params p) {
  __shared__ uint32_t s_row0[kSlabRows];
  __shared__ uint32_t s_row1[kSlabRows];
  __shared__ float s_lamy[kSlabRows];

  const uint32_t img = blockIdx.x / p.slabs;
  const uint32_t slab = blockIdx.x - img * p.slabs;
  const preba_img_t e = p.table[img];
  if (!entry_ok(e, p.pixels_bytes)) {
    if (threadIdx.x == 0) report(p.status, PREBA_ERR_BAD_TABLE);
    return;
  }
  const uint32_t C = p.C;
  uint64_t rh, rw;
  if (e.h <= e.w) {
    rh = p.S;
    rw = static_cast<uint64_t>(p.S) * e.w / e.h;
  } else {
    rw = p.S;
    rh = static_cast<uint64_t>(p.S) * e.h / e.w;
  }
  const uint64_t top = (rh - C) / 2, left = (rw - C) / 2;
  const uint32_t k_first = slab * kSlabRows;
  const uint32_t rows = min(kSlabRows, C - k_first);
  const uint32_t pitch = 3 * e.w;

  if (threadIdx.x < rows) {
    const Tap t = axis_tap(e.h, rh, top, k_first + threadIdx.x);
    s_row0[threadIdx.x] = t.i0 * pitch;
    s_row1[threadIdx.x] = t.i1 * pitch;
    s_lamy[threadIdx.x] = t.lam;
  }
  __syncthreads();

  const uint8_t* __restrict__ src = p.pixels + e.offset;
  OutT* __restrict__ out = static_cast<OutT*>(p.out);
  const size_t plane = static_cast<size_t>(C) * C;
  const size_t img_base = static_cast<size_t>(img) * 3 * plane;

  for (uint32_t j = threadIdx.x; j < C; j += kThreads) {
    const Tap tx = axis_tap(e.w, rw, left, j);
    const uint32_t c0 = 3 * tx.i0, c1 = 3 * tx.i1;
    for (uint32_t r = 0; r < rows; ++r) {
      const uint8_t* row0 = src + s_row0[r];
      const uint8_t* row1 = src + s_row1[r];
      const float ly = s_lamy[r];
      const size_t o = img_base + static_cast<size_t>(k_first + r) * C + j;
#pragma unroll
      for (int ch = 0; ch < 3; ++ch) {
        const float p00 = __ldg(row0 + c0 + ch), p01 = __ldg(row0 + c1 + ch);
        const float p10 = __ldg(row1 + c0 + ch), p11 = __ldg(row1 + c1 + ch);
        const float h0 = fmaf(tx.lam, p01 - p00, p00);
        const float h1 = fmaf(tx.lam, p11 - p10, p10);
        const float v = fmaf(ly, h1 - h0, h0);
        store_out(out + o + ch * plane, fmaf(v, p.a[ch], p.b[ch]));
      }
    }
  }
}

thread_local int g_last_cuda_error = 0;

int check_args(const uint8_t* pixels, uint64_t pixels_bytes, const void* table, uint32_t n,
               const void* out, uint64_t out_bytes, uint32_t out_size, uint32_t resize_short,
               const float mean[3], const float std[3], int out_dtype) {
  if (!pixels || !table || !out || !mean || !std || n == 0) return PREBA_ERR_INVALID_ARG;
  if (!dtype_ok(out_dtype) || out_size == 0 || resize_short < out_size ||
      resize_short > PREBA_MAX_RESIZE)
    return PREBA_ERR_INVALID_ARG;
  for (int c = 0; c < 3; ++c)
    if (!std::isfinite(mean[c]) || !std::isfinite(std[c]) || std[c] == 0.0f)
      return PREBA_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(pixels) % 16 || reinterpret_cast<uintptr_t>(out) % 16 ||
      reinterpret_cast<uintptr_t>(table) % 8)
    return PREBA_ERR_INVALID_ARG;
  const uint64_t need = static_cast<uint64_t>(n) * 3ull * out_size * out_size *
                        (out_dtype == PREBA_F16 ? 2u : 4u);
  if (out_bytes < need) return PREBA_ERR_BUFFER_TOO_SMALL;
  if (pixels_bytes == 0) return PREBA_ERR_BUFFER_TOO_SMALL;
  return PREBA_OK;
}

int check_table(const preba_img_t* t, uint32_t n, uint64_t pixels_bytes) {
  for (uint32_t i = 0; i < n; ++i) {
    if (!dims_ok(t[i].h, t[i].w) || t[i].offset % PREBA_PACK_ALIGN) return PREBA_ERR_BAD_TABLE;
    const uint64_t bytes = 3ull * t[i].h * t[i].w;
    if (t[i].offset > pixels_bytes || bytes > pixels_bytes - t[i].offset)
      return PREBA_ERR_BAD_TABLE;
  }
  return PREBA_OK;
}

int launch(const Params& p, int out_dtype, cudaStream_t stream) {
  const uint64_t blocks = static_cast<uint64_t>(p.n) * p.slabs;
  if (blocks > 0x7fffffffull) return PREBA_ERR_INVALID_ARG;
  const dim3 grid(static_cast<unsigned>(blocks));
  if (out_dtype == PREBA_F16)
    preba_gather_kernel<__half><<<grid, kThreads, 0, stream>>>(p);
  else
    preba_gather_kernel<float><<<grid, kThreads, 0, stream>>>(p);
  const cudaError_t err = cudaGetLastError();
  if (err != cudaSuccess) {
    g_last_cuda_error = static_cast<int>(err);
    return PREBA_ERR_CUDA;
  }
  return PREBA_OK;
}

Params make_params(const uint8_t* pixels, uint64_t pixels_bytes, const preba_img_t* table,
                   uint32_t n, void* out, int32_t* status, uint32_t out_size,
                   uint32_t resize_short, const float mean[3], const float std[3]) {
  Params p;
  p.pixels = pixels;
  p.pixels_bytes = pixels_bytes;
  p.table = table;
  p.out = out;
  p.status = status;
  p.n = n;
  p.C = out_size;
  p.S = resize_short;
  p.slabs = (out_size + kSlabRows - 1) / kSlabRows;
  for (int c = 0; c < 3; ++c) {
    const double sd = static_cast<double>(std[c]);
    p.a[c] = static_cast<float>(1.0 / (255.0 * sd));
    p.b[c] = static_cast<float>(-static_cast<double>(mean[c]) / sd);
  }
  return p;
}

}  // namespace preba

extern "C" int preba_preprocess(const preba_batch_t* batch, uint32_t out_size,
                                uint32_t resize_short, const float mean[3], const float std[3],
                                int out_dtype, void* stream) {
  using namespace preba;
  if (!batch) return PREBA_ERR_INVALID_ARG;
  int rc = check_args(batch->pixels, batch->pixels_bytes, batch->table, batch->n, batch->out,
                      batch->out_bytes, out_size, resize_short, mean, std, out_dtype);
  if (rc != PREBA_OK) return rc;
  if (batch->table_host) {
    rc = check_table(batch->table_host, batch->n, batch->pixels_bytes);
    if (rc != PREBA_OK) return rc;
  }
  const Params p = make_params(batch->pixels, batch->pixels_bytes, batch->table, batch->n,
                               batch->out, batch->status, out_size, resize_short, mean, std);
  return launch(p, out_dtype, static_cast<cudaStream_t>(stream));
}

extern "C" int preba_preprocess_host(const preba_host_batch_t* b, uint32_t out_size,
                                     uint32_t resize_short, const float mean[3],
                                     const float std[3], int out_dtype, void* stream) {
  using namespace preba;
  if (!b || !b->packed_host || !b->table_host || !b->out_host || !b->dev_table)
    return PREBA_ERR_INVALID_ARG;
  int rc = check_args(b->dev_pixels, b->packed_bytes, b->dev_table, b->n, b->dev_out,
                      b->out_bytes, out_size, resize_short, mean, std, out_dtype);
  if (rc != PREBA_OK) return rc;
  rc = check_table(b->table_host, b->n, b->packed_bytes);
  if (rc != PREBA_OK) return rc;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const uint64_t need = static_cast<uint64_t>(b->n) * 3ull * out_size * out_size *
                        (out_dtype == PREBA_F16 ? 2u : 4u);
  cudaError_t err = cudaMemcpyAsync(b->dev_pixels, b->packed_host, b->packed_bytes,
                                    cudaMemcpyHostToDevice, s);
  if (err == cudaSuccess)
    err = cudaMemcpyAsync(b->dev_table, b->table_host, sizeof(preba_img_t) * b->n,
                          cudaMemcpyHostToDevice, s);
  if (err != cudaSuccess) {
    g_last_cuda_error = static_cast<int>(err);
    return PREBA_ERR_CUDA;
  }
  const Params p = make_params(b->dev_pixels, b->packed_bytes, b->dev_table, b->n, b->dev_out,
                               b->dev_status, out_size, resize_short, mean, std);
  rc = launch(p, out_dtype, s);
  if (rc != PREBA_OK) return rc;
  err = cudaMemcpyAsync(b->out_host, b->dev_out, need, cudaMemcpyDeviceToHost, s);
  if (err != cudaSuccess) {
    g_last_cuda_error = static_cast<int>(err);
    return PREBA_ERR_CUDA;
  }
  return PREBA_OK;
}

extern "C" int preba_last_cuda_error(void) { return preba::g_last_cuda_error; }
