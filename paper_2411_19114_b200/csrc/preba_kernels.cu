// Fused resize -> center crop -> normalise -> HWC->NCHW for a ragged batch (sm_100a).
//
// One launch per batch, persistent grid.  Every warp works on its own: it claims a task
// (a slab of output rows of one image, up to 224 output columns wide), reads the image's
// {offset, h, w} from the device table, derives the sampling grid in exact integers and
// streams the tapped source rows into its private shared-memory ring with bulk asynchronous
// copies (one per row, 16-byte aligned, completion counted on an mbarrier).  While a group
// of rows is in flight the warp computes on the previous one: per staged row each lane
// interpolates horizontally for its seven output columns and keeps the previous row's
// result in registers; whenever both source rows of an output row have passed, it
// interpolates vertically, applies the normalising multiply-add, converts and stores
// planar output.  The copy stream runs ahead across task boundaries, so a warp's next task
// is already arriving while it finishes the current one.  Nothing but the input bytes and
// the output tensor touches device memory; warps never wait for one another.
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <atomic>
#include <cmath>

#include "preba.h"
#include "preba_internal.h"

namespace preba {

#ifndef PREBA_WARPS_PER_CTA
#define PREBA_WARPS_PER_CTA 4
#endif
#ifndef PREBA_CTAS_PER_SM
#define PREBA_CTAS_PER_SM 6
#endif
#ifndef PREBA_SLAB_ROWS
#define PREBA_SLAB_ROWS 16
#endif
#ifndef PREBA_GROUP_BYTES
#define PREBA_GROUP_BYTES 2816
#endif
#ifndef PREBA_GROUP_ROWS
#define PREBA_GROUP_ROWS 2
#endif

constexpr int kWarpsPerCta = PREBA_WARPS_PER_CTA;
constexpr int kThreads = 32 * kWarpsPerCta;
constexpr int kCtasPerSm = PREBA_CTAS_PER_SM;
constexpr uint32_t kLaneCols = 7;                  // output columns per lane
constexpr uint32_t kTaskCols = 32 * kLaneCols;     // 224 output columns per task
constexpr uint32_t kSlabRows = PREBA_SLAB_ROWS;    // output rows per task (one lane per row)
constexpr uint32_t kMaxList = 2 * 32;              // distinct source rows of a slab
constexpr uint32_t kGroups = 2;                    // ring: one group computed, one in flight
constexpr uint32_t kGroupBytes = PREBA_GROUP_BYTES;
constexpr uint32_t kGroupRows = PREBA_GROUP_ROWS;  // rows per group at most
constexpr uint32_t kSpinLimit = 1u << 20;          // bounded waits: give up, report, leave
static_assert(kSlabRows >= 1 && kSlabRows <= 32, "one lane per output row of a slab");
static_assert(kGroupBytes % 16 == 0, "bulk copies need 16-byte aligned destinations");

enum TaskKind : uint32_t { kEnd = 0, kStream = 1, kGather = 2, kSkip = 3 };

struct Params {
  const uint8_t* pixels;
  uint64_t pixels_bytes;
  const preba_img_t* table;
  void* out;
  int32_t* status;
  uint32_t* sched;      // two zeroed words for dynamic task claims, or NULL for static turns
  uint32_t n;
  uint32_t C;           // crop side
  uint32_t S;           // resized shorter side
  uint32_t slabs;       // slabs per image
  uint32_t col_blocks;  // column blocks per image
  uint32_t tasks;       // n * slabs * col_blocks
  float a[3];           // 1 / (255 * std_c)
  float b[3];           // -mean_c / std_c
};

// A task as its warp sees it, in the warp's shared memory.
struct TaskMeta {
  uint32_t kind;
  uint32_t img, k0, rows_out, col0;
  uint32_t w, h, rw, rh;  // input size, resized size
  uint32_t xmin;          // first source column staged
  uint32_t stride;        // bytes between staged rows of a group
  uint32_t rows_per_group;
  uint32_t n_list;        // distinct source rows of the slab, ascending
  uint32_t copy_bytes;    // tapped bytes of a staged row
  uint64_t src;           // byte offset of the image in the pixel buffer
  uint32_t info[kMaxList];  // per listed row: low byte = byte skew of the staged row,
                            // next byte = output rows completed by this row (<= 32)
  uint32_t lam[32];         // per output row: weight of the lower source row (float bits);
                            // sign bit set when both taps are the same row
  uint32_t row[kMaxList];   // per listed row: source row index
};

struct __align__(16) WarpShared {
  uint8_t ring[kGroups][kGroupBytes];
  TaskMeta meta;
  uint64_t full[kGroups];
};

// Taps and weight of one crop-window index along one axis: the source coordinate
// ((origin + j) + 1/2) * in / r - 1/2, clamped to [0, in - 1], as num / den with
// num = (2X + 1) * in - r and den = 2r.  i0 = floor(num / den) and the remainder are exact
// integers; the weight is the remainder over den in fp32.
struct Tap {
  uint32_t i0;
  uint32_t i1;
  float lam;
};

struct Axis {
  uint32_t in;      // source length
  uint32_t r;       // resized length
  uint32_t origin;  // crop origin on the resized axis
  uint32_t den;     // 2r
  uint32_t hi;      // (in - 1) * den when it fits 32 bits
  float rden;       // 1 / den
  bool small;       // every numerator fits 32 bits and den is exact in fp32
};

__device__ __forceinline__ Axis make_axis(uint32_t in, uint32_t r, uint32_t origin, uint32_t c) {
  Axis a;
  a.in = in;
  a.r = r;
  a.origin = origin;
  a.den = 2 * r;  // r <= 2^29
  const uint64_t top = (2ull * (origin + c) + 1) * in;  // above every numerator of the crop
  a.small = top < (1ull << 32) && a.den < (1u << 24);
  // the clamp at the far end: (in - 1) * den, or "never" when that exceeds every numerator
  const uint64_t hi = static_cast<uint64_t>(in - 1) * a.den;
  a.hi = hi < (1ull << 32) ? static_cast<uint32_t>(hi) : 0xffffffffu;
  a.rden = 1.0f / static_cast<float>(a.den);
  return a;
}

__device__ __forceinline__ Tap axis_tap(const Axis& a, uint32_t j) {
  Tap t;
  if (a.small) {
    // quotient from an fp32 estimate (relative error < 2^-21, so off by at most one),
    // made exact by the integer remainder
    const uint32_t pos = (2 * (a.origin + j) + 1) * a.in;
    uint32_t num = pos > a.r ? pos - a.r : 0;
    num = min(num, a.hi);
    uint32_t q = __float2uint_rz(__uint2float_rz(num) * a.rden);
    int32_t rem = static_cast<int32_t>(num - q * a.den);
    if (rem < 0) {
      --q;
      rem += static_cast<int32_t>(a.den);
    } else if (rem >= static_cast<int32_t>(a.den)) {
      ++q;
      rem -= static_cast<int32_t>(a.den);
    }
    t.i0 = q;
    t.lam = static_cast<float>(rem) * a.rden;
  } else {
    const uint64_t den = 2ull * a.r;
    const uint64_t pos = (2 * (static_cast<uint64_t>(a.origin) + j) + 1) * a.in;  // < 2^46
    uint64_t num = pos > a.r ? pos - a.r : 0;
    const uint64_t hi = static_cast<uint64_t>(a.in - 1) * den;
    num = num < hi ? num : hi;
    const uint64_t q = num / den;
    t.i0 = static_cast<uint32_t>(q);
    t.lam = static_cast<float>(num - q * den) / static_cast<float>(den);
  }
  t.i1 = t.i0 + 1 < a.in ? t.i0 + 1 : a.in - 1;
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

// Orders this thread's earlier shared-memory reads before later asynchronous-copy writes.
__device__ __forceinline__ void fence_async_shared() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// Three consecutive aligned words of shared memory.
__device__ __forceinline__ void lds32x3(uint32_t addr, uint32_t& w0, uint32_t& w1, uint32_t& w2) {
  asm volatile(
      "ld.shared.u32 %0, [%3];\n\t"
      "ld.shared.u32 %1, [%3+4];\n\t"
      "ld.shared.u32 %2, [%3+8];"
      : "=r"(w0), "=r"(w1), "=r"(w2)
      : "r"(addr));
}

// ---- arithmetic ---------------------------------------------------------------------------------

// Byte `idx` of x as 2^23 + byte: the byte dropped into the mantissa of 8388608.0f.
template <int idx>
__device__ __forceinline__ float byte_biased(uint32_t x) {
  return __uint_as_float(__byte_perm(x, 0x4B000000u, 0x7440 + idx));
}

// Horizontal interpolation at shared-memory byte address x (pixel x0, then x0 + 1); x is
// unaligned: three aligned words are read and shifted.
__device__ __forceinline__ void hlerp_row(uint32_t x, float lam, float h[3]) {
  const uint32_t addr = x & ~3u;
  const uint32_t sh = x << 3;  // the funnel shift takes it modulo 32
  uint32_t w0, w1, w2;
  lds32x3(addr, w0, w1, w2);
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

// Columns of a lane inside a task: three adjacent pairs 64 columns apart, then one single.
__device__ __forceinline__ uint32_t lane_col(uint32_t lane, uint32_t m) {
  return m < 6 ? 2 * lane + 64 * (m >> 1) + (m & 1) : 192 + lane;
}

// What a lane keeps for the task it computes on.
struct Lane {
  uint32_t off[kLaneCols];  // byte offset of the first tap in a staged row (before its skew)
  float lam[kLaneCols];     // weight of the second tap
  uint32_t valid;           // bit m: column m exists
};

// Normalised output value from the two horizontal results around it.
__device__ __forceinline__ float blend(float prev, float cur, float ly, float a, float b) {
  return fmaf(fmaf(ly, cur - prev, prev), a, b);
}

// Column group g of a lane: g < 3 is the pair (2g, 2g + 1), g == 3 the single column 6.
// Stores the group's outputs of one row; q points at column 2 * lane of plane 0.
template <typename OutT, bool FULL, int G>
__device__ __forceinline__ void store_group(OutT* __restrict__ q, uint32_t plane, uint32_t lane,
                                            const float (&prev)[kLaneCols][3],
                                            const float (&c0)[3], const float (&c1)[3], float ly,
                                            const float (&na)[3], const float (&nb)[3],
                                            uint32_t valid) {
#pragma unroll
  for (int ch = 0; ch < 3; ++ch, q += plane) {
    if (G < 3) {
      const float o0 = blend(prev[2 * G][ch], c0[ch], ly, na[ch], nb[ch]);
      const float o1 = blend(prev[2 * G + 1][ch], c1[ch], ly, na[ch], nb[ch]);
      if (FULL) {
        *reinterpret_cast<typename Pack<OutT>::Vec*>(q + 64 * G) = Pack<OutT>::pair(o0, o1);
      } else {
        if ((valid >> (2 * G)) & 1u) q[64 * G] = Pack<OutT>::one(o0);
        if ((valid >> (2 * G + 1)) & 1u) q[64 * G + 1] = Pack<OutT>::one(o1);
      }
    } else {
      const float o0 = blend(prev[6][ch], c0[ch], ly, na[ch], nb[ch]);
      if (FULL || ((valid >> 6) & 1u)) q[192 - lane] = Pack<OutT>::one(o0);
    }
  }
}

// One staged row: per column group the horizontal pass, then the `e` output rows the row
// completes (weights from lam[], sign bit = both taps are this row), then the row's result
// becomes `prev` of the next step.
template <typename OutT, bool FULL>
__device__ __forceinline__ void step_row(uint32_t base, uint32_t e, const uint32_t* lam,
                                         OutT* __restrict__ q, uint32_t C, uint32_t plane,
                                         uint32_t lane, const Lane& ln,
                                         float (&prev)[kLaneCols][3], const float (&na)[3],
                                         const float (&nb)[3]) {
#pragma unroll
  for (int g = 0; g < 4; ++g) {
    const int m0 = g < 3 ? 2 * g : 6, m1 = g < 3 ? 2 * g + 1 : 6;
    float a0[3], a1[3] = {0.f, 0.f, 0.f};
    hlerp_row(base + ln.off[m0], ln.lam[m0], a0);
    if (g < 3) hlerp_row(base + ln.off[m1], ln.lam[m1], a1);
    OutT* qq = q;
    for (uint32_t j = 0; j < e; ++j, qq += C) {
      const uint32_t lbits = lam[j];
      const float ly = __uint_as_float(lbits & 0x7fffffffu);
      if (lbits >> 31) {  // both taps are this row: the result is the row itself
#pragma unroll
        for (int ch = 0; ch < 3; ++ch) {
          prev[m0][ch] = a0[ch];
          if (g < 3) prev[m1][ch] = a1[ch];
        }
      }
      if (g == 0) store_group<OutT, FULL, 0>(qq, plane, lane, prev, a0, a1, ly, na, nb, ln.valid);
      if (g == 1) store_group<OutT, FULL, 1>(qq, plane, lane, prev, a0, a1, ly, na, nb, ln.valid);
      if (g == 2) store_group<OutT, FULL, 2>(qq, plane, lane, prev, a0, a1, ly, na, nb, ln.valid);
      if (g == 3) store_group<OutT, FULL, 3>(qq, plane, lane, prev, a0, a1, ly, na, nb, ln.valid);
    }
#pragma unroll
    for (int ch = 0; ch < 3; ++ch) {
      prev[m0][ch] = a0[ch];
      if (g < 3) prev[m1][ch] = a1[ch];
    }
  }
}

// ---- task preparation: geometry of a slab into the warp's meta buffer --------------------------

// Fills `m` for task `task`; returns its kind.  All lanes take part.
__device__ __forceinline__ uint32_t prepare(const Params& p, uint32_t task, TaskMeta& m,
                                            uint32_t lane) {
  const uint32_t C = p.C;
  const uint32_t per_img = p.slabs * p.col_blocks;
  const uint32_t img = task / per_img;
  const uint32_t rest = task - img * per_img;
  const uint32_t slab = rest / p.col_blocks;
  const uint32_t cb = rest - slab * p.col_blocks;
  const preba_img_t e = p.table[img];
  uint32_t kind = kSkip;
  if (entry_ok(e, p.pixels_bytes)) {
    uint32_t rh, rw;
    if (e.h <= e.w) {
      rh = p.S;
      rw = static_cast<uint32_t>(static_cast<uint64_t>(p.S) * e.w / e.h);
    } else {
      rw = p.S;
      rh = static_cast<uint32_t>(static_cast<uint64_t>(p.S) * e.h / e.w);
    }
    const uint32_t top = (rh - C) / 2, left = (rw - C) / 2;
    const uint32_t k0 = slab * kSlabRows;
    const uint32_t rows_out = min(kSlabRows, C - k0);
    const uint32_t col0 = cb * kTaskCols;
    const uint32_t cols = min(kTaskCols, C - col0);
    const Axis ax = make_axis(e.w, rw, left, C);
    const Tap tf = axis_tap(ax, col0);
    const Tap tl = axis_tap(ax, col0 + cols - 1);
    const uint32_t xmin = tf.i0;
    const uint32_t copy_px = tl.i1 - xmin + 1;
    // a lane reads 12 bytes from the word holding its first tap, which may be the last
    // staged pixel: leave room for one more pixel and the word overshoot
    const uint32_t stride = (15 + 3 * copy_px + 3 + 12 + 15) & ~15u;
    const uint32_t rpg = min(kGroupRows, kGroupBytes / stride);
    const uint64_t end16 = (e.offset + 3ull * e.h * e.w + 15) & ~15ull;
    kind = (rpg >= 1 && end16 <= p.pixels_bytes) ? kStream : kGather;

    // rows of the slab: taps, then the ascending list of distinct source rows
    const bool active = lane < rows_out;
    const Axis ay = make_axis(e.h, rh, top, C);
    Tap ty = {0, 0, 0.f};
    if (active) ty = axis_tap(ay, k0 + lane);
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
    const uint32_t n_list = __shfl_sync(0xffffffffu, incl, 31);
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
    if (active) m.lam[lane] = __float_as_uint(ty.lam) | (ty.i1 == ty.i0 ? 0x80000000u : 0u);
    __syncwarp();
    for (uint32_t i = lane; i < n_list; i += 32)
      m.info[i] |= (3u * (m.row[i] * e.w + xmin)) & 15u;
    if (lane == 0) {
      m.img = img;
      m.k0 = k0;
      m.rows_out = rows_out;
      m.col0 = col0;
      m.w = e.w;
      m.h = e.h;
      m.rw = rw;
      m.rh = rh;
      m.xmin = xmin;
      m.stride = stride;
      m.rows_per_group = rpg;
      m.n_list = n_list;
      m.copy_bytes = 3 * copy_px;
      m.src = e.offset;
    }
  } else {
    if (lane == 0) report(p.status, PREBA_ERR_BAD_TABLE);
  }
  if (lane == 0) m.kind = kind;
  __syncwarp();
  return kind;
}

// ---- the warp program ---------------------------------------------------------------------------------

// Issues the copies of one group of listed rows [first, first + cnt) into ring slot `slot`.
__device__ __forceinline__ void issue_group(WarpShared& ws, uint32_t slot, uint32_t first,
                                            uint32_t cnt, const uint8_t* base, uint32_t pitch,
                                            uint32_t copy_bytes, uint32_t stride, uint32_t lane) {
  const uint32_t bar = smem_addr(&ws.full[slot]);
  if (lane < kGroupRows) {
    if (lane < cnt) {
      const uint8_t* src = base + static_cast<size_t>(ws.meta.row[first + lane]) * pitch;
      const uintptr_t s = reinterpret_cast<uintptr_t>(src);
      const uintptr_t s0 = s & ~static_cast<uintptr_t>(15);
      const uint32_t bytes =
          static_cast<uint32_t>(((s + copy_bytes + 15) & ~static_cast<uintptr_t>(15)) - s0);
      fence_async_shared();
      mbar_arrive_expect_tx(bar, bytes);
      bulk_copy_g2s(smem_addr(&ws.ring[slot][lane * stride]), reinterpret_cast<const void*>(s0),
                    bytes, bar);
    } else {
      mbar_arrive(bar);
    }
  }
}

template <typename OutT>
__device__ __forceinline__ void warp_main(const Params& p, WarpShared& ws, uint32_t lane,
                                          uint32_t gwarp, uint32_t nwarps) {
  const uint32_t C = p.C;
  const uint32_t plane = C * C;
  const float na[3] = {p.a[0], p.a[1], p.a[2]};
  const float nb[3] = {p.b[0], p.b[1], p.b[2]};
  const TaskMeta& m = ws.meta;
  uint32_t groups_done = 0;  // groups waited for so far: ring slot and barrier phase
  bool failed = false;
  Lane ln;
  float prev[kLaneCols][3];
#pragma unroll
  for (int c = 0; c < static_cast<int>(kLaneCols); ++c)
#pragma unroll
    for (int ch = 0; ch < 3; ++ch) prev[c][ch] = 0.f;

  // a warp's first task is its own index; later ones come from the shared counter (claimed
  // when a task ends) or, without scratch, every nwarps-th task
  for (uint32_t task = gwarp; task < p.tasks && !failed;) {
    const uint32_t kind = prepare(p, task, ws.meta, lane);
    if (kind != kSkip) {
      const uint32_t w = m.w, rw = m.rw, col0 = m.col0, xmin = m.xmin;
      const Axis ax = make_axis(w, rw, (rw - C) / 2, C);
      ln.valid = 0;
#pragma unroll
      for (int c = 0; c < static_cast<int>(kLaneCols); ++c) {
        const uint32_t j = col0 + lane_col(lane, c);
        if (j < C) ln.valid |= 1u << c;
        const Tap t = axis_tap(ax, j < C ? j : C - 1);
        ln.off[c] = 3 * (t.i0 - xmin);
        ln.lam[c] = t.lam;
      }
      const bool full = (C & 1u) == 0 && __all_sync(0xffffffffu, ln.valid == 0x7fu);
      // column 2 * lane of the task's first output row, plane 0
      OutT* q_out = static_cast<OutT*>(p.out) + static_cast<size_t>(m.img) * 3 * plane +
                    (m.k0 * C + col0 + 2 * lane);
      if (kind == kStream) {
        const uint32_t n_list = m.n_list, rpg = m.rows_per_group, stride = m.stride;
        const uint8_t* base = p.pixels + m.src + 3 * xmin;
        const uint32_t pitch = 3 * w, copy_bytes = m.copy_bytes;
        // two groups in flight, then one more each time a group has been computed
        issue_group(ws, groups_done % kGroups, 0, min(rpg, n_list), base, pitch, copy_bytes, stride,
                    lane);
        if (rpg < n_list)
          issue_group(ws, (groups_done + 1) % kGroups, rpg, min(rpg, n_list - rpg), base, pitch,
                      copy_bytes, stride, lane);
        uint32_t t_out = 0;
        for (uint32_t row = 0; row < n_list; row += rpg) {
          const uint32_t slot = groups_done % kGroups;
          if (!mbar_wait(smem_addr(&ws.full[slot]), (groups_done / kGroups) & 1)) {
            failed = true;
            break;
          }
          ++groups_done;
          const uint32_t cnt = min(rpg, n_list - row);
          uint32_t row_addr = smem_addr(&ws.ring[slot][0]);
          for (uint32_t r = 0; r < cnt; ++r, row_addr += stride) {
            const uint32_t info = m.info[row + r];
            const uint32_t e = (info >> 8) & 0xffu;
            if (full)
              step_row<OutT, true>(row_addr + (info & 0xffu), e, &m.lam[t_out], q_out, C, plane,
                                   lane, ln, prev, na, nb);
            else
              step_row<OutT, false>(row_addr + (info & 0xffu), e, &m.lam[t_out], q_out, C, plane,
                                    lane, ln, prev, na, nb);
            t_out += e;
            q_out += e * C;
          }
          __syncwarp();  // every lane is done with the slot before it is refilled
          const uint32_t next = row + kGroups * rpg;
          if (next < n_list)
            issue_group(ws, slot, next, min(rpg, n_list - next), base, pitch, copy_bytes, stride,
                        lane);
        }
        if (failed) {
          // copies already issued may still be landing in the ring: wait for them (bounded)
          // before the CTA can retire
          for (uint32_t g = 0; g < kGroups; ++g)
            (void)mbar_wait(smem_addr(&ws.full[(groups_done + g) % kGroups]),
                            ((groups_done + g) / kGroups) & 1);
        }
      } else {
        // direct path: taps straight from global memory (footprint too wide for the ring)
        const uint8_t* __restrict__ src = p.pixels + m.src + 3 * xmin;
        const size_t pitch = 3 * static_cast<size_t>(w);
        const uint32_t h = m.h, rh = m.rh, k0 = m.k0, rows_out = m.rows_out;
        const Axis ay = make_axis(h, rh, (rh - C) / 2, C);
        for (uint32_t t = 0; t < rows_out; ++t, q_out += C) {
          const Tap ty = axis_tap(ay, k0 + t);
          const uint8_t* r0 = src + ty.i0 * pitch;
          const uint8_t* r1 = src + ty.i1 * pitch;
#pragma unroll
          for (int c = 0; c < static_cast<int>(kLaneCols); ++c) {
            // the right neighbour is read only where it carries weight (it exists then)
            const uint32_t nbr = ln.lam[c] > 0.f ? 3u : 0u;
            float h1[3];
#pragma unroll
            for (int ch = 0; ch < 3; ++ch) {
              float a = __ldg(r0 + ln.off[c] + ch), b = __ldg(r0 + ln.off[c] + nbr + ch);
              prev[c][ch] = fmaf(ln.lam[c], b - a, a);
              a = __ldg(r1 + ln.off[c] + ch), b = __ldg(r1 + ln.off[c] + nbr + ch);
              h1[ch] = fmaf(ln.lam[c], b - a, a);
            }
            OutT* qc = q_out + (c < 6 ? 64 * (c >> 1) + (c & 1) : 192 - static_cast<int>(lane));
            if ((ln.valid >> c) & 1u) {
#pragma unroll
              for (int ch = 0; ch < 3; ++ch)
                qc[static_cast<size_t>(ch) * plane] =
                    Pack<OutT>::one(blend(prev[c][ch], h1[ch], ty.lam, na[ch], nb[ch]));
            }
          }
        }
      }
    }
    __syncwarp();  // the meta buffer is free again
    if (p.sched) {
      uint32_t got = 0;
      if (lane == 0) got = atomicAdd(&p.sched[0], 1u);
      task = nwarps + __shfl_sync(0xffffffffu, got, 0);
    } else {
      task = task + nwarps >= task ? task + nwarps : p.tasks;
    }
  }

  if (failed && lane == 0) report(p.status, PREBA_ERR_TIMEOUT);
  // the last warp out leaves the claim counters at zero for the next launch
  if (p.sched && lane == 0) {
    __threadfence();
    if (atomicAdd(&p.sched[1], 1u) == nwarps - 1) {
      p.sched[0] = 0;
      p.sched[1] = 0;
    }
  }
}

template <typename OutT>
__global__ void __launch_bounds__(kThreads, kCtasPerSm) preba_fused_kernel(const Params p) {
  __shared__ WarpShared sm[kWarpsPerCta];
  const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  WarpShared& ws = sm[warp];
  if (lane == 0) {
    for (uint32_t g = 0; g < kGroups; ++g) mbar_init(smem_addr(&ws.full[g]), kGroupRows);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncwarp();
  warp_main<OutT>(p, ws, lane, blockIdx.x * kWarpsPerCta + warp, gridDim.x * kWarpsPerCta);
}

// ---- tile kernel: a CTA stages the rows of a slab once, threads evaluate pixels --------------------

#ifndef PREBA_TILE_ROWS
#define PREBA_TILE_ROWS 16
#endif
#ifndef PREBA_TILE_BYTES
#define PREBA_TILE_BYTES 32768
#endif
#ifndef PREBA_TILE_CTAS
#define PREBA_TILE_CTAS 5
#endif

constexpr uint32_t kTileRows = PREBA_TILE_ROWS;    // output rows per tile
constexpr uint32_t kTileCols = 224;                // output columns per tile
constexpr uint32_t kTilePairs = kTileCols / 2;     // a thread owns two adjacent columns
constexpr uint32_t kTileThreads = 2 * kTilePairs;  // even and odd rows of a pass
constexpr uint32_t kTileBytes = PREBA_TILE_BYTES;  // staged rows
static_assert(kTileRows <= 32 && (kTileRows & (kTileRows - 1)) == 0, "power of two, <= 32");
static_assert(kTileThreads % 32 == 0, "whole warps");

struct __align__(16) TileShared {
  uint8_t rows[kTileBytes];
  uint64_t full;             // completion of a pass's copies
  uint32_t kind;             // kStream, kGather or kSkip
  uint32_t pass_rows;        // output rows of the current pass
  uint32_t img, k0, rows_out, col0, w, h, rw, rh, xmin;
  uint64_t src;              // byte offset of the image in the pixel buffer
  uint32_t a0[kTileRows];    // per output row of the pass: shared address of the first
  uint32_t a1[kTileRows];    //   tapped byte of its upper / lower source row
  uint32_t ly[kTileRows];    // weight of the lower row (float bits)
  uint32_t list[32];         // source rows of the pass (producer's scratch)
  uint32_t xoff[kTileCols];  // per output column: byte offset of its first tap in a staged row
  float xlam[kTileCols];     //   and the weight of the second tap
};

// Builds the pass [r0, r0 + rows) of the tile: tables and copies.  Warp 0, all lanes.
// Returns false if the pass does not fit the staging buffer.
__device__ __forceinline__ bool tile_pass(const Params& p, TileShared& ts, const Axis& ay,
                                          uint32_t r0, uint32_t rows, uint32_t stride,
                                          uint32_t copy_bytes, const uint8_t* base, uint32_t pitch,
                                          uint32_t lane, uint32_t* n_list_out) {
  const bool active = lane < rows;
  Tap ty = {0, 0, 0.f};
  if (active) ty = axis_tap(ay, ts.k0 + r0 + lane);
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
  const uint32_t n_list = __shfl_sync(0xffffffffu, incl, 31);
  *n_list_out = n_list;
  if (n_list > 32 || n_list * stride > kTileBytes) return false;
  const uint32_t excl = incl - cnt;
  if (new0) ts.list[excl] = ty.i0;
  if (new1) ts.list[excl + (new0 ? 1u : 0u)] = ty.i1;
  // slot of the lower row = last listed so far; the upper row is the one before it
  // unless both taps coincide
  const uint32_t s1 = incl - 1;
  const uint32_t s0 = ty.i1 == ty.i0 ? s1 : s1 - 1;
  const uint32_t ring = smem_addr(&ts.rows[0]);
  if (active) {
    const uint32_t skew0 = (3u * (ty.i0 * ts.w + ts.xmin)) & 15u;
    const uint32_t skew1 = (3u * (ty.i1 * ts.w + ts.xmin)) & 15u;
    ts.a0[lane] = ring + s0 * stride + skew0;
    ts.a1[lane] = ring + s1 * stride + skew1;
    ts.ly[lane] = __float_as_uint(ty.lam);
  }
  __syncwarp();
  const uint32_t bar = smem_addr(&ts.full);
  // one arrival per lane: a copy (with its byte count) or a plain arrival
  if (lane < n_list) {
    const uint8_t* src = base + static_cast<size_t>(ts.list[lane]) * pitch;
    const uintptr_t s = reinterpret_cast<uintptr_t>(src);
    const uintptr_t sa = s & ~static_cast<uintptr_t>(15);
    const uint32_t bytes =
        static_cast<uint32_t>(((s + copy_bytes + 15) & ~static_cast<uintptr_t>(15)) - sa);
    fence_async_shared();
    mbar_arrive_expect_tx(bar, bytes);
    bulk_copy_g2s(ring + lane * stride, reinterpret_cast<const void*>(sa), bytes, bar);
  } else {
    mbar_arrive(bar);
  }
  return true;
}

template <typename OutT>
__global__ void __launch_bounds__(kTileThreads, PREBA_TILE_CTAS) preba_tile_kernel(const Params p) {
  __shared__ TileShared ts;
  const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t C = p.C;
  const uint32_t plane = C * C;

  // which tile
  const uint32_t per_img = p.slabs * p.col_blocks;
  const uint32_t img = blockIdx.x / per_img;
  const uint32_t rest = blockIdx.x - img * per_img;
  const uint32_t slab = rest / p.col_blocks;
  const uint32_t cb = rest - slab * p.col_blocks;
  const preba_img_t e = p.table[img];
  if (!entry_ok(e, p.pixels_bytes)) {
    if (tid == 0) report(p.status, PREBA_ERR_BAD_TABLE);
    return;
  }
  uint32_t rh, rw;
  if (e.h <= e.w) {
    rh = p.S;
    rw = static_cast<uint32_t>(static_cast<uint64_t>(p.S) * e.w / e.h);
  } else {
    rw = p.S;
    rh = static_cast<uint32_t>(static_cast<uint64_t>(p.S) * e.h / e.w);
  }
  const uint32_t k0 = slab * kTileRows;
  const uint32_t rows_out = min(kTileRows, C - k0);
  const uint32_t col0 = cb * kTileCols;
  const uint32_t cols = min(kTileCols, C - col0);
  const Axis ax = make_axis(e.w, rw, (rw - C) / 2, C);
  const Tap tf = axis_tap(ax, col0);
  const Tap tl = axis_tap(ax, col0 + cols - 1);
  const uint32_t xmin = tf.i0;
  const uint32_t copy_px = tl.i1 - xmin + 1;
  // a thread reads 12 bytes from the word holding its first tap, which may be the last
  // staged pixel: leave room for one more pixel and the word overshoot
  const uint32_t stride = (15 + 3 * copy_px + 3 + 12 + 15) & ~15u;
  const uint64_t end16 = (e.offset + 3ull * e.h * e.w + 15) & ~15ull;
  const bool stream = 2 * stride <= kTileBytes && end16 <= p.pixels_bytes;

  if (tid == 0) {
    mbar_init(smem_addr(&ts.full), 32);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    ts.k0 = k0;
    ts.w = e.w;
    ts.xmin = xmin;
  }
  // column taps of the tile, one per thread
  if (tid < cols) {
    const Tap t = axis_tap(ax, col0 + tid);
    ts.xoff[tid] = 3 * (t.i0 - xmin);
    ts.xlam[tid] = t.lam;
  }
  __syncthreads();

  const uint32_t cp = tid % kTilePairs, rg = tid / kTilePairs;  // column pair, row parity
  const uint32_t jA = 2 * cp;
  const bool validA = jA < cols, validB = jA + 1 < cols;
  const uint32_t offA = ts.xoff[validA ? jA : 0], offB = ts.xoff[validB ? jA + 1 : 0];
  const float lamA = ts.xlam[validA ? jA : 0], lamB = ts.xlam[validB ? jA + 1 : 0];
  const bool pair_ok = (C & 1u) == 0 && validB;
  const float na[3] = {p.a[0], p.a[1], p.a[2]};
  const float nb[3] = {p.b[0], p.b[1], p.b[2]};
  OutT* out_img = static_cast<OutT*>(p.out) + static_cast<size_t>(img) * 3 * plane + col0 + jA;
  const Axis ay = make_axis(e.h, rh, (rh - C) / 2, C);

  if (stream) {
    const uint8_t* base = p.pixels + e.offset + 3 * xmin;
    const uint32_t pitch = 3 * e.w;
    uint32_t pass_rows = kTileRows;  // shrinks (by halves) until a pass fits the buffer
    uint32_t pass = 0;
    for (uint32_t r0 = 0; r0 < rows_out; ++pass) {
      if (warp == 0) {
        uint32_t n_list = 0;
        uint32_t rows = min(pass_rows, rows_out - r0);
        while (!tile_pass(p, ts, ay, r0, rows, stride, 3 * copy_px, base, pitch, lane, &n_list)) {
          pass_rows >>= 1;  // two rows always fit (checked above), so this ends at >= 1
          rows = min(pass_rows, rows_out - r0);
        }
        if (lane == 0) ts.pass_rows = rows;
      }
      __syncthreads();
      const uint32_t rows = ts.pass_rows;
      if (!mbar_wait(smem_addr(&ts.full), pass & 1)) {
        if (lane == 0) report(p.status, PREBA_ERR_TIMEOUT);
        return;  // (the copies land in this CTA's memory or not at all: nothing to undo)
      }
      for (uint32_t r = rg; r < rows; r += 2) {
        const uint32_t a0 = ts.a0[r], a1 = ts.a1[r];
        const float ly = __uint_as_float(ts.ly[r]);
        float tA[3], bA[3], tB[3], bB[3];
        hlerp_row(a0 + offA, lamA, tA);
        hlerp_row(a1 + offA, lamA, bA);
        hlerp_row(a0 + offB, lamB, tB);
        hlerp_row(a1 + offB, lamB, bB);
        OutT* q = out_img + static_cast<size_t>(k0 + r0 + r) * C;
#pragma unroll
        for (int ch = 0; ch < 3; ++ch, q += plane) {
          const float oA = blend(tA[ch], bA[ch], ly, na[ch], nb[ch]);
          const float oB = blend(tB[ch], bB[ch], ly, na[ch], nb[ch]);
          if (pair_ok) {
            *reinterpret_cast<typename Pack<OutT>::Vec*>(q) = Pack<OutT>::pair(oA, oB);
          } else {
            if (validA) q[0] = Pack<OutT>::one(oA);
            if (validB) q[1] = Pack<OutT>::one(oB);
          }
        }
      }
      r0 += rows;
      if (r0 < rows_out) __syncthreads();  // everyone is done with the buffer
    }
  } else {
    // direct path: taps straight from global memory (a row pair exceeds the buffer)
    const uint8_t* __restrict__ src = p.pixels + e.offset + 3 * xmin;
    const size_t pitch = 3 * static_cast<size_t>(e.w);
    const uint32_t nA = lamA > 0.f ? 3u : 0u, nB = lamB > 0.f ? 3u : 0u;
    for (uint32_t r = rg; r < rows_out; r += 2) {
      const Tap ty = axis_tap(ay, k0 + r);
      const uint8_t* r0p = src + ty.i0 * pitch;
      const uint8_t* r1p = src + ty.i1 * pitch;
      OutT* q = out_img + static_cast<size_t>(k0 + r) * C;
#pragma unroll
      for (int ch = 0; ch < 3; ++ch, q += plane) {
        // the right neighbour is read only where it carries weight (it exists then)
        float a = __ldg(r0p + offA + ch), b = __ldg(r0p + offA + nA + ch);
        const float tA = fmaf(lamA, b - a, a);
        a = __ldg(r1p + offA + ch), b = __ldg(r1p + offA + nA + ch);
        const float bA = fmaf(lamA, b - a, a);
        a = __ldg(r0p + offB + ch), b = __ldg(r0p + offB + nB + ch);
        const float tB = fmaf(lamB, b - a, a);
        a = __ldg(r1p + offB + ch), b = __ldg(r1p + offB + nB + ch);
        const float bB = fmaf(lamB, b - a, a);
        if (validA) q[0] = Pack<OutT>::one(blend(tA, bA, ty.lam, na[ch], nb[ch]));
        if (validB) q[1] = Pack<OutT>::one(blend(tB, bB, ty.lam, na[ch], nb[ch]));
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
  const uint64_t tasks = static_cast<uint64_t>(n) * ((out_size + kSlabRows - 1) / kSlabRows) *
                         ((out_size + kTaskCols - 1) / kTaskCols);
  if (tasks > 0x7fffffffull) return PREBA_ERR_INVALID_ARG;
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
// The answer depends on the device and the kernel only; it is computed once per device and
// output type and kept (a benign race: concurrent first calls store the same value).
int resident_ctas(int out_dtype, cudaError_t* err) {
  constexpr int kMaxDevices = 64;
  static std::atomic<int> cache[2][kMaxDevices];
  int dev = 0;
  *err = cudaGetDevice(&dev);
  if (*err != cudaSuccess) return 0;
  const int kind = out_dtype == PREBA_F16 ? 1 : 0;
  if (dev >= 0 && dev < kMaxDevices) {
    const int known = cache[kind][dev].load(std::memory_order_relaxed);
    if (known > 0) return known;
  }
  int sms = 0, per_sm = 0;
  *err = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (*err != cudaSuccess) return 0;
  if (kind == 1)
    *err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, preba_fused_kernel<__half>,
                                                         kThreads, 0);
  else
    *err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, preba_fused_kernel<float>,
                                                         kThreads, 0);
  if (*err != cudaSuccess) return 0;
  const int resident = sms * (per_sm > 0 ? per_sm : 1);
  if (dev >= 0 && dev < kMaxDevices) cache[kind][dev].store(resident, std::memory_order_relaxed);
  return resident;
}

#ifndef PREBA_KERNEL
#define PREBA_KERNEL 1
#endif

int launch(const Params& p, int out_dtype, cudaStream_t stream) {
  cudaError_t err = cudaSuccess;
#if PREBA_KERNEL == 1
  {
    Params q = p;
    q.slabs = (p.C + kTileRows - 1) / kTileRows;
    q.col_blocks = (p.C + kTileCols - 1) / kTileCols;
    const uint64_t blocks = static_cast<uint64_t>(p.n) * q.slabs * q.col_blocks;
    if (blocks > 0x7fffffffull) return PREBA_ERR_INVALID_ARG;
    if (out_dtype == PREBA_F16)
      preba_tile_kernel<__half><<<static_cast<unsigned>(blocks), kTileThreads, 0, stream>>>(q);
    else
      preba_tile_kernel<float><<<static_cast<unsigned>(blocks), kTileThreads, 0, stream>>>(q);
    err = cudaGetLastError();
    if (err != cudaSuccess) {
      g_last_cuda_error = static_cast<int>(err);
      return PREBA_ERR_CUDA;
    }
    return PREBA_OK;
  }
#endif
  const int resident = resident_ctas(out_dtype, &err);
  if (err == cudaSuccess) {
    const uint32_t want = (p.tasks + kWarpsPerCta - 1) / kWarpsPerCta;
    const uint32_t blocks = want < static_cast<uint32_t>(resident) ? want : resident;
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
                   uint32_t n, void* out, int32_t* status, uint32_t* scratch, uint32_t out_size,
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
  p.sched = scratch;
  p.slabs = (out_size + kSlabRows - 1) / kSlabRows;
  p.col_blocks = (out_size + kTaskCols - 1) / kTaskCols;
  p.tasks = static_cast<uint32_t>(static_cast<uint64_t>(n) * p.slabs * p.col_blocks);
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
  if (reinterpret_cast<uintptr_t>(batch->scratch) % 16) return PREBA_ERR_INVALID_ARG;
  if (batch->table_host) {
    rc = check_table(batch->table_host, batch->n, batch->pixels_bytes);
    if (rc != PREBA_OK) return rc;
  }
  const Params p = make_params(batch->pixels, batch->pixels_bytes, batch->table, batch->n,
                               batch->out, batch->status, batch->scratch, out_size, resize_short,
                               mean, std);
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
  if (reinterpret_cast<uintptr_t>(b->dev_scratch) % 16) return PREBA_ERR_INVALID_ARG;
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
                               b->dev_status, b->dev_scratch, out_size, resize_short, mean, std);
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
