// Fused resize -> center crop -> normalise -> HWC->NCHW for a ragged batch (sm_100a).
//
// One launch per batch.  The grid is persistent: each CTA walks over tiles, a tile being a
// slab of output rows (times a block of up to 256 output columns) of one image.  Inside a
// CTA one producer warp reads the image's {offset, h, w} from the device table, derives
// the sampling grid in exact integers, and streams the tapped source rows into a ring of
// shared-memory stages with bulk asynchronous copies (one per row, 16-byte aligned,
// completion counted on an mbarrier).  Four consumer warps follow the ring: per staged
// row every thread interpolates horizontally for its two output columns, keeps the
// previous row's result in registers, and emits an output row whenever both of its source
// rows have passed -- vertical interpolation, normalising multiply-add, conversion and a
// vectorised planar store.  The ring keeps filling across tile boundaries, so the copies
// of the next tile are in flight while the current one is computed; nothing but the
// input bytes and the output tensor touches device memory.
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <cmath>

#include "preba.h"
#include "preba_internal.h"

namespace preba {

constexpr int kConsumerWarps = 4;
constexpr int kConsumerThreads = kConsumerWarps * 32;
constexpr int kThreads = kConsumerThreads + 32;  // + one producer warp
constexpr uint32_t kTileCols = 2 * kConsumerThreads;  // two output columns per consumer thread
constexpr uint32_t kMaxSlabRows = 32;                 // one producer lane per output row
constexpr uint32_t kMaxList = 2 * kMaxSlabRows;       // distinct source rows of a slab
constexpr int kStages = 4;
constexpr uint32_t kStageBytes = 6144;
constexpr uint32_t kMaxRowsPerStage = 8;
constexpr uint32_t kSpinLimit = 1u << 20;  // bounded waits: give up, report, leave

enum TileKind : uint32_t { kEnd = 0, kStream = 1, kGather = 2, kSkip = 3 };

struct Params {
  const uint8_t* pixels;
  uint64_t pixels_bytes;
  const preba_img_t* table;
  void* out;
  int32_t* status;
  uint32_t n;
  uint32_t C;          // crop side
  uint32_t S;          // resized shorter side
  uint32_t slab_rows;  // output rows per tile, <= kMaxSlabRows
  uint32_t slabs;      // slabs per image
  uint32_t col_blocks; // column blocks per image
  uint32_t tiles;      // n * slabs * col_blocks
  float a[3];          // 1 / (255 * std_c)
  float b[3];          // -mean_c / std_c
};

// What the producer tells the consumers about a tile.
struct TileMeta {
  uint32_t kind;
  uint32_t img, k0, rows_out, col0;
  uint32_t w, rw, left;  // x axis: input width, resized width, crop origin
  uint32_t xmin;         // first source column staged
  uint32_t stride;       // bytes between staged rows of a stage
  uint32_t rows_per_stage;
  uint32_t n_list;       // distinct source rows of the slab, ascending
  uint64_t src;          // byte offset of the image in the pixel buffer
  uint32_t info[kMaxList];    // per listed row: low byte = byte skew of the staged row,
                              // next byte = output rows completed by this row
  uint32_t lam[kMaxSlabRows]; // per output row: weight of the lower source row (float bits);
                              // sign bit set when both taps are the same row
  uint32_t row[kMaxList];     // per listed row: source row index
  uint32_t y0[kMaxSlabRows];  // per output row: tap rows (direct path)
  uint32_t y1[kMaxSlabRows];
};

// Taps and weight of one crop-window index along one axis: the source coordinate
// ((origin + j) + 1/2) * in / r - 1/2, clamped to [0, in - 1], as num / den with
// num = (2X + 1) * in - r and den = 2r.
struct Tap {
  uint32_t i0;
  uint32_t i1;
  float lam;
};

__device__ __forceinline__ Tap axis_tap(uint32_t in, uint32_t r, uint32_t origin, uint32_t j) {
  const uint64_t X = static_cast<uint64_t>(origin) + j;
  const uint64_t den = 2ull * r;
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

// ---- shared-memory barriers and bulk copies (PTX) -------------------------------------------

__device__ __forceinline__ uint32_t smem_addr(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}

__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
               : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}

// Waits for the phase with the given parity to complete; false if the limit ran out.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  for (uint32_t it = 0; it < kSpinLimit; ++it)
    if (mbar_try_wait(bar, parity)) return true;
  return false;
}

// Global -> shared bulk copy; both addresses and the size are multiples of 16 bytes.
__device__ __forceinline__ void bulk_copy_g2s(uint32_t dst, const void* src, uint32_t bytes,
                                              uint32_t bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
      ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
      : "memory");
}

__device__ __forceinline__ uint32_t lds32(uint32_t addr) {
  uint32_t v;
  asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
  return v;
}

// ---- arithmetic ---------------------------------------------------------------------------------

// Byte `idx` of x as 2^23 + byte: the byte dropped into the mantissa of 8388608.0f.
template <int idx>
__device__ __forceinline__ float byte_biased(uint32_t x) {
  return __uint_as_float(__byte_perm(x, 0x4B000000u, 0x7440 + idx));
}

// Horizontal interpolation of one staged row at byte offset `off` (pixel x0, then x0+1).
__device__ __forceinline__ void hlerp_row(uint32_t row_addr, uint32_t off, float lam, float h[3]) {
  const uint32_t addr = row_addr + (off & ~3u);
  const uint32_t sh = (off & 3u) * 8u;
  const uint32_t w0 = lds32(addr), w1 = lds32(addr + 4), w2 = lds32(addr + 8);
  const uint32_t lo = __funnelshift_r(w0, w1, sh);  // R0 G0 B0 R1
  const uint32_t hi = __funnelshift_r(w1, w2, sh);  // G1 B1 .. ..
  const float a0 = byte_biased<0>(lo), a1 = byte_biased<1>(lo), a2 = byte_biased<2>(lo);
  const float b0 = byte_biased<3>(lo), b1 = byte_biased<0>(hi), b2 = byte_biased<1>(hi);
  h[0] = fmaf(lam, b0 - a0, a0 - 8388608.0f);
  h[1] = fmaf(lam, b1 - a1, a1 - 8388608.0f);
  h[2] = fmaf(lam, b2 - a2, a2 - 8388608.0f);
}

template <typename OutT>
struct Pack;
template <>
struct Pack<float> {
  using Vec = float2;
  static __device__ __forceinline__ Vec pair(float x, float y) { return make_float2(x, y); }
  static __device__ __forceinline__ float one(float x) { return x; }
};
template <>
struct Pack<__half> {
  using Vec = __half2;
  static __device__ __forceinline__ Vec pair(float x, float y) { return __floats2half2_rn(x, y); }
  static __device__ __forceinline__ __half one(float x) { return __float2half_rn(x); }
};

// Vertical interpolation, normalisation and store of one output row for two columns.
template <typename OutT>
__device__ __forceinline__ void emit_row(OutT* __restrict__ dst, size_t plane, float ly,
                                         const float hpA[3], const float hcA[3],
                                         const float hpB[3], const float hcB[3],
                                         const Params& p, bool pair_ok, bool validA, bool validB) {
#pragma unroll
  for (int ch = 0; ch < 3; ++ch) {
    const float vA = fmaf(ly, hcA[ch] - hpA[ch], hpA[ch]);
    const float vB = fmaf(ly, hcB[ch] - hpB[ch], hpB[ch]);
    const float oA = fmaf(vA, p.a[ch], p.b[ch]);
    const float oB = fmaf(vB, p.a[ch], p.b[ch]);
    OutT* q = dst + ch * plane;
    if (pair_ok) {
      *reinterpret_cast<typename Pack<OutT>::Vec*>(q) = Pack<OutT>::pair(oA, oB);
    } else {
      if (validA) q[0] = Pack<OutT>::one(oA);
      if (validB) q[1] = Pack<OutT>::one(oB);
    }
  }
}

struct __align__(16) Shared {
  uint8_t ring[kStages][kStageBytes];
  TileMeta meta[2];
  uint64_t full[kStages];
  uint64_t empty[kStages];
  uint64_t meta_full[2];
  uint64_t meta_empty[2];
};

// ---- producer warp ---------------------------------------------------------------------------------

__device__ __forceinline__ void produce(const Params& p, Shared& sm, uint32_t lane) {
  const uint32_t C = p.C;
  uint32_t fills = 0;  // stages filled so far by this CTA
  bool failed = false;
  for (uint32_t it = 0; !failed; ++it) {
    const uint32_t mb = it & 1;
    TileMeta& m = sm.meta[mb];
    if (it >= 2 && !mbar_wait(smem_addr(&sm.meta_empty[mb]), ((it >> 1) - 1) & 1)) {
      failed = true;
      break;
    }
    const uint64_t tile = static_cast<uint64_t>(blockIdx.x) + static_cast<uint64_t>(it) * gridDim.x;
    if (tile >= p.tiles) {
      if (lane == 0) m.kind = kEnd;
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_addr(&sm.meta_full[mb]));
      break;
    }
    const uint32_t per_img = p.slabs * p.col_blocks;
    const uint32_t img = static_cast<uint32_t>(tile / per_img);
    const uint32_t rest = static_cast<uint32_t>(tile - static_cast<uint64_t>(img) * per_img);
    const uint32_t slab = rest / p.col_blocks;
    const uint32_t cb = rest - slab * p.col_blocks;
    const preba_img_t e = p.table[img];
    const bool ok = entry_ok(e, p.pixels_bytes);
    uint32_t kind = kSkip;
    uint32_t n_list = 0, rps = 0, stride = 0, xmin = 0, copy_px = 0;
    if (ok) {
      uint32_t rh, rw;
      if (e.h <= e.w) {
        rh = p.S;
        rw = static_cast<uint32_t>(static_cast<uint64_t>(p.S) * e.w / e.h);
      } else {
        rw = p.S;
        rh = static_cast<uint32_t>(static_cast<uint64_t>(p.S) * e.h / e.w);
      }
      const uint32_t top = (rh - C) / 2, left = (rw - C) / 2;
      const uint32_t k0 = slab * p.slab_rows;
      const uint32_t rows_out = min(p.slab_rows, C - k0);
      const uint32_t col0 = cb * kTileCols;
      const uint32_t cols = min(kTileCols, C - col0);
      const Tap tf = axis_tap(e.w, rw, left, col0);
      const Tap tl = axis_tap(e.w, rw, left, col0 + cols - 1);
      xmin = tf.i0;
      copy_px = tl.i1 - xmin + 1;
      // a consumer reads 12 bytes from the word holding its first tap, which may be the
      // last staged pixel: leave room for one more pixel and the word overshoot
      stride = (15 + 3 * copy_px + 3 + 12 + 15) & ~15u;
      rps = min(kMaxRowsPerStage, kStageBytes / stride);
      const uint64_t end16 = (e.offset + 3ull * e.h * e.w + 15) & ~15ull;
      kind = (rps >= 1 && end16 <= p.pixels_bytes) ? kStream : kGather;

      // rows of the slab: taps, then the ascending list of distinct source rows
      const bool active = lane < rows_out;
      Tap ty = {0, 0, 0.f};
      if (active) ty = axis_tap(e.h, rh, top, k0 + lane);
      const uint32_t y1_prev = __shfl_up_sync(0xffffffffu, ty.i1, 1);
      const bool new0 = active && (lane == 0 || ty.i0 > y1_prev);
      const bool new1 = active && ty.i1 != ty.i0 && (lane == 0 || ty.i1 > y1_prev);
      const uint32_t cnt = (new0 ? 1u : 0u) + (new1 ? 1u : 0u);
      uint32_t incl = cnt;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const uint32_t v = __shfl_up_sync(0xffffffffu, incl, d);
        if (lane >= static_cast<uint32_t>(d)) incl += v;
      }
      n_list = __shfl_sync(0xffffffffu, incl, 31);
      const uint32_t excl = incl - cnt;
      if (new0) m.row[excl] = ty.i0;
      if (new1) m.row[excl + (new0 ? 1u : 0u)] = ty.i1;
      m.info[lane] = 0;
      m.info[lane + 32] = 0;
      __syncwarp();
      // the row that completes output row `lane` is the last one listed so far
      const uint32_t key = active ? incl - 1 : 0x80000000u + lane;
      const uint32_t peers = __match_any_sync(0xffffffffu, key);
      if (active && lane == static_cast<uint32_t>(__ffs(peers) - 1))
        m.info[key] = static_cast<uint32_t>(__popc(peers)) << 8;
      if (active) {
        m.lam[lane] = __float_as_uint(ty.lam) | (ty.i1 == ty.i0 ? 0x80000000u : 0u);
        m.y0[lane] = ty.i0;
        m.y1[lane] = ty.i1;
      }
      __syncwarp();
      for (uint32_t i = lane; i < n_list; i += 32)
        m.info[i] |= (3u * (m.row[i] * e.w + xmin)) & 15u;
      if (lane == 0) {
        m.img = img;
        m.k0 = k0;
        m.rows_out = rows_out;
        m.col0 = col0;
        m.w = e.w;
        m.rw = rw;
        m.left = left;
        m.xmin = xmin;
        m.stride = stride;
        m.rows_per_stage = rps;
        m.n_list = n_list;
        m.src = e.offset;
      }
    } else if (lane == 0) {
      report(p.status, PREBA_ERR_BAD_TABLE);
    }
    if (lane == 0) m.kind = kind;
    __syncwarp();
    if (lane == 0) mbar_arrive(smem_addr(&sm.meta_full[mb]));

    if (kind == kStream) {
      const uint8_t* img_base = p.pixels + e.offset;
      const uint32_t pitch = 3 * e.w;
      for (uint32_t base = 0; base < n_list; base += rps) {
        const uint32_t stage = fills % kStages;
        if (fills >= kStages &&
            !mbar_wait(smem_addr(&sm.empty[stage]), ((fills / kStages) - 1) & 1)) {
          failed = true;
          break;
        }
        const uint32_t cnt = min(rps, n_list - base);
        const uint32_t bar = smem_addr(&sm.full[stage]);
        if (lane < cnt) {
          const uint8_t* src = img_base + static_cast<size_t>(m.row[base + lane]) * pitch + 3 * xmin;
          const uintptr_t s = reinterpret_cast<uintptr_t>(src);
          const uintptr_t s0 = s & ~static_cast<uintptr_t>(15);
          const uint32_t bytes =
              static_cast<uint32_t>(((s + 3 * copy_px + 15) & ~static_cast<uintptr_t>(15)) - s0);
          mbar_arrive_expect_tx(bar, bytes);
          bulk_copy_g2s(smem_addr(&sm.ring[stage][lane * stride]),
                        reinterpret_cast<const void*>(s0), bytes, bar);
        } else {
          mbar_arrive(bar);
        }
        ++fills;
      }
    }
  }
  if (failed) {
    if (lane == 0) report(p.status, PREBA_ERR_TIMEOUT);
    // copies already issued may still be landing in this CTA's shared memory: wait for
    // them (bounded) before the CTA can retire
    const uint32_t first = fills > kStages ? fills - kStages : 0;
    for (uint32_t f = first; f < fills; ++f)
      (void)mbar_wait(smem_addr(&sm.full[f % kStages]), (f / kStages) & 1);
  }
}

// ---- consumer warps -----------------------------------------------------------------------------------

template <typename OutT>
__device__ __forceinline__ void consume(const Params& p, Shared& sm, uint32_t tid, uint32_t lane) {
  const uint32_t C = p.C;
  const size_t plane = static_cast<size_t>(C) * C;
  const bool even = (C & 1u) == 0;
  uint32_t drains = 0;  // stages consumed so far by this CTA
  for (uint32_t it = 0;; ++it) {
    const uint32_t mb = it & 1;
    if (!mbar_wait(smem_addr(&sm.meta_full[mb]), (it >> 1) & 1)) {
      if (lane == 0) report(p.status, PREBA_ERR_TIMEOUT);
      return;
    }
    const TileMeta& m = sm.meta[mb];
    const uint32_t kind = m.kind;
    if (kind == kEnd) return;
    if (kind != kSkip) {
      const uint32_t w = m.w, rw = m.rw, left = m.left;
      const uint32_t rows_out = m.rows_out;
      const uint32_t jA = m.col0 + 2 * tid;
      const bool validA = jA < C, validB = jA + 1 < C;
      const bool pair_ok = even && validB;
      const Tap tA = axis_tap(w, rw, left, validA ? jA : m.col0);
      const Tap tB = axis_tap(w, rw, left, validB ? jA + 1 : (validA ? jA : m.col0));
      OutT* dst = static_cast<OutT*>(p.out) +
                  (static_cast<size_t>(m.img) * 3 * C + m.k0) * C + jA;
      if (kind == kStream) {
        const uint32_t n_list = m.n_list, rps = m.rows_per_stage, stride = m.stride;
        const uint32_t offA = 3 * (tA.i0 - m.xmin), offB = 3 * (tB.i0 - m.xmin);
        float hpA[3] = {0.f, 0.f, 0.f}, hcA[3] = {0.f, 0.f, 0.f};
        float hpB[3] = {0.f, 0.f, 0.f}, hcB[3] = {0.f, 0.f, 0.f};
        uint32_t t_out = 0;
        for (uint32_t base = 0; base < n_list; base += rps) {
          const uint32_t stage = drains % kStages;
          if (!mbar_wait(smem_addr(&sm.full[stage]), (drains / kStages) & 1)) {
            if (lane == 0) report(p.status, PREBA_ERR_TIMEOUT);
            return;
          }
          const uint32_t cnt = min(rps, n_list - base);
          uint32_t row_addr = smem_addr(&sm.ring[stage][0]);
          for (uint32_t r = 0; r < cnt; ++r, row_addr += stride) {
            const uint32_t info = m.info[base + r];
            const uint32_t skew = info & 0xffu;
#pragma unroll
            for (int ch = 0; ch < 3; ++ch) {
              hpA[ch] = hcA[ch];
              hpB[ch] = hcB[ch];
            }
            hlerp_row(row_addr, offA + skew, tA.lam, hcA);
            hlerp_row(row_addr, offB + skew, tB.lam, hcB);
            for (uint32_t e = info >> 8; e > 0; --e, ++t_out) {
              const uint32_t lbits = m.lam[t_out];
              float ly = __uint_as_float(lbits);
              if (lbits >> 31) {  // both taps are this row
#pragma unroll
                for (int ch = 0; ch < 3; ++ch) {
                  hpA[ch] = hcA[ch];
                  hpB[ch] = hcB[ch];
                }
                ly = 0.f;
              }
              emit_row<OutT>(dst, plane, ly, hpA, hcA, hpB, hcB, p, pair_ok, validA, validB);
              dst += C;
            }
          }
          __syncwarp();
          if (lane == 0) mbar_arrive(smem_addr(&sm.empty[stage]));
          ++drains;
        }
      } else {  // direct path: taps straight from global memory
        const uint8_t* __restrict__ src = p.pixels + m.src;
        const size_t pitch = 3 * static_cast<size_t>(w);
        const uint32_t cA0 = 3 * tA.i0, cA1 = 3 * tA.i1, cB0 = 3 * tB.i0, cB1 = 3 * tB.i1;
        for (uint32_t t = 0; t < rows_out; ++t, dst += C) {
          const uint8_t* r0 = src + m.y0[t] * pitch;
          const uint8_t* r1 = src + m.y1[t] * pitch;
          const float ly = __uint_as_float(m.lam[t] & 0x7fffffffu);
          float h0A[3], h1A[3], h0B[3], h1B[3];
#pragma unroll
          for (int ch = 0; ch < 3; ++ch) {
            float a = __ldg(r0 + cA0 + ch), b = __ldg(r0 + cA1 + ch);
            h0A[ch] = fmaf(tA.lam, b - a, a);
            a = __ldg(r1 + cA0 + ch), b = __ldg(r1 + cA1 + ch);
            h1A[ch] = fmaf(tA.lam, b - a, a);
            a = __ldg(r0 + cB0 + ch), b = __ldg(r0 + cB1 + ch);
            h0B[ch] = fmaf(tB.lam, b - a, a);
            a = __ldg(r1 + cB0 + ch), b = __ldg(r1 + cB1 + ch);
            h1B[ch] = fmaf(tB.lam, b - a, a);
          }
          emit_row<OutT>(dst, plane, ly, h0A, h1A, h0B, h1B, p, pair_ok, validA, validB);
        }
      }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(smem_addr(&sm.meta_empty[mb]));
  }
}

template <typename OutT>
__global__ void __launch_bounds__(kThreads) preba_fused_kernel(const Params p) {
  __shared__ Shared sm;
  const uint32_t tid = threadIdx.x, lane = tid & 31;
  if (tid == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(smem_addr(&sm.full[s]), 32);               // every producer lane arrives
      mbar_init(smem_addr(&sm.empty[s]), kConsumerWarps);  // one arrival per consumer warp
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_addr(&sm.meta_full[b]), 1);
      mbar_init(smem_addr(&sm.meta_empty[b]), kConsumerWarps);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (tid >= kConsumerThreads)
    produce(p, sm, lane);
  else
    consume<OutT>(p, sm, tid, lane);
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
  const uint64_t tiles = static_cast<uint64_t>(n) * ((out_size + 7) / 8) *
                         ((out_size + kTileCols - 1) / kTileCols);
  if (tiles > 0x7fffffffull) return PREBA_ERR_INVALID_ARG;
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

// Resident CTAs of the fused kernel on the current device (grid of a persistent launch).
int resident_ctas(int out_dtype, cudaError_t* err) {
  int dev = 0, sms = 0, per_sm = 0;
  *err = cudaGetDevice(&dev);
  if (*err != cudaSuccess) return 0;
  *err = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (*err != cudaSuccess) return 0;
  if (out_dtype == PREBA_F16)
    *err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, preba_fused_kernel<__half>,
                                                         kThreads, 0);
  else
    *err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, preba_fused_kernel<float>,
                                                         kThreads, 0);
  if (*err != cudaSuccess) return 0;
  return sms * (per_sm > 0 ? per_sm : 1);
}

int launch(const Params& p, int out_dtype, cudaStream_t stream) {
  cudaError_t err = cudaSuccess;
  const int resident = resident_ctas(out_dtype, &err);
  if (err == cudaSuccess) {
    const uint32_t blocks = p.tiles < static_cast<uint32_t>(resident) ? p.tiles : resident;
    if (out_dtype == PREBA_F16)
      preba_fused_kernel<__half><<<blocks, kThreads, 0, stream>>>(p);
    else
      preba_fused_kernel<float><<<blocks, kThreads, 0, stream>>>(p);
    err = cudaGetLastError();
  }
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
  p.slab_rows = 16;
  p.slabs = (out_size + p.slab_rows - 1) / p.slab_rows;
  p.col_blocks = (out_size + kTileCols - 1) / kTileCols;
  p.tiles = static_cast<uint32_t>(static_cast<uint64_t>(n) * p.slabs * p.col_blocks);
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
