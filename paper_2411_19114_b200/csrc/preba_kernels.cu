// Fused resize -> center crop -> normalise -> HWC->NCHW for a ragged batch (sm_100a).
//
// One launch per batch, persistent grid.  Every warp works on its own: it claims a task
// (a slab of output rows of one image, up to 224 output columns wide), reads the image's
// {offset, h, w} from the device table, derives the sampling grid in exact integers and
// streams the tapped source rows into its private shared-memory ring with bulk asynchronous
// copies (one per row, 16-byte aligned, completion counted on an mbarrier).  While a group
// of rows is in flight the warp computes on the previous one: per staged row each lane
// interpolates horizontally for its seven output columns in exact integers (two taps times
// their integer weights, a 16-bit-by-8-bit two-way dot product per channel) and keeps the
// previous row's result in registers; whenever both source rows of an output row have
// passed, it interpolates vertically in fp32, applies the normalising multiply-add (which
// also divides by the weights' common denominator), converts and stores planar output.  The copy stream runs ahead across task boundaries, so a warp's next task
// is already arriving while it finishes the current one.  Nothing but the input bytes and
// the output tensor touches device memory; warps never wait for one another.
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <atomic>
#include <cmath>
#include <cstdint>
#include <vector>

#include "preba.h"
#include "preba_internal.h"

namespace preba {

#ifndef PREBA_WARPS_PER_CTA
#define PREBA_WARPS_PER_CTA 4
#endif
#ifndef PREBA_CTAS_PER_SM
#define PREBA_CTAS_PER_SM 4
#endif
#ifndef PREBA_SLAB_ROWS
#define PREBA_SLAB_ROWS 32
#endif
#ifndef PREBA_GROUP_BYTES
#define PREBA_GROUP_BYTES 4608
#endif

constexpr int kWarpsPerCta = PREBA_WARPS_PER_CTA;
constexpr int kThreads = 32 * kWarpsPerCta;
constexpr int kCtasPerSm = PREBA_CTAS_PER_SM;
constexpr uint32_t kLaneCols = 7;                  // output columns per lane
constexpr uint32_t kTaskCols = 32 * kLaneCols;     // 224 output columns per task
constexpr uint32_t kSlabRows = PREBA_SLAB_ROWS;    // output rows per task (one lane per row)
#ifndef PREBA_MIN_SLAB_ROWS
#define PREBA_MIN_SLAB_ROWS 4
#endif
constexpr uint32_t kMinSlabRows = PREBA_MIN_SLAB_ROWS;  // smallest slab a small batch is cut into
constexpr uint32_t kMaxList = 2 * 32;              // distinct source rows of a slab
#ifndef PREBA_GROUPS
#define PREBA_GROUPS 2
#endif
#ifndef PREBA_GROUP_ROWS
#define PREBA_GROUP_ROWS 6
#endif
constexpr uint32_t kGroups = PREBA_GROUPS;         // ring: one group computed, the rest in flight
constexpr uint32_t kGroupBytes = PREBA_GROUP_BYTES;
constexpr uint32_t kGroupRows = PREBA_GROUP_ROWS;  // rows per group at most
constexpr uint32_t kMetaBufs = 3;                  // the copy stream is at most two tasks ahead
constexpr uint32_t kSpinLimit = 1u << 20;          // bounded waits: give up, report, leave
static_assert(kSlabRows >= 1 && kSlabRows <= 32, "one lane per output row of a slab");
static_assert(kGroupBytes % 16 == 0, "bulk copies need 16-byte aligned destinations");

enum TaskKind : uint32_t { kEnd = 0, kStream = 1, kGather = 2, kSkip = 3 };

// What leaves the vertical stage.  kFloat: the interpolated value, normalised (fp32
// arithmetic).  kRoundFloat: the value rounded to the nearest integer, ties up, decided in
// exact integer arithmetic, then normalised.  kU8: that integer itself as uint8, HWC.
enum Mode : int { kFloat = 0, kRoundFloat = 1, kU8 = 2 };

struct Params {
  const uint8_t* pixels;
  uint64_t pixels_bytes;
  const preba_img_t* table;
  void* out;
  int32_t* status;
  uint32_t* sched;      // two zeroed words for dynamic task claims, or NULL for static turns
  const uint32_t* crop; // per image (top, left) of the window on the resized grid, or NULL: centre
  uint32_t n;
  uint32_t C;           // crop side
  uint32_t S;           // resized shorter side
  uint32_t slab_rows;   // output rows per task: 32, or fewer (down to 4) in a launch that runs
                        // alone, so that its busiest warp has the least to do
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
  uint32_t top, left;     // first row and column of the window on the resized grid
  // rounded modes: the value of an output pixel is num / dd with dd = den_x * den_y
  uint32_t deny2;         // 2 * den_y
  uint32_t dd;            // den_x * den_y
  uint32_t magic;         // reciprocal of 2 * dd (see Quant)
  uint32_t shift;         // k - 1 when the reciprocal is exact, else kNoShift
  uint32_t pad;
  uint64_t src;           // byte offset of the image in the pixel buffer
  uint32_t info[kMaxList];  // per listed row: low byte = byte skew of the staged row,
                            // next byte = output rows completed by this row
  uint32_t lam[32];         // per output row: weight of the lower source row (float bits);
                            // 1.0f when both taps are the same row (the row just staged):
                            // staged values are whole numbers below 2^24, so
                            // prev + 1 * (cur - prev) is cur exactly, whatever prev holds
  uint32_t row[kMaxList];   // per listed row: source row index
};

struct __align__(16) WarpShared {
  uint8_t ring[kGroups][kGroupBytes];
  TaskMeta meta[kMetaBufs];
  uint64_t full[kGroups];
};

// Taps and weight of one crop-window index along one axis: the source coordinate
// ((origin + j) + 1/2) * in / r - 1/2, clamped to [0, in - 1], as num / den with
// num = (2X + 1) * in - r and den = 2r.  i0 = floor(num / den) and the remainder are exact
// integers; the weight is the remainder over den in fp32.
struct Tap {
  uint32_t i0;
  uint32_t i1;
  uint32_t rem;  // num mod den (filled by the 32-bit path only)
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

// The tap when a.small holds: straight-line 32-bit code, so that several taps interleave.
// The quotient comes from an fp32 estimate (relative error < 2^-21, so off by at most one)
// and is made exact by the integer remainder.
__device__ __forceinline__ Tap axis_tap_small(const Axis& a, uint32_t j) {
  Tap t;
  const uint32_t pos = (2 * (a.origin + j) + 1) * a.in;
  uint32_t num = max(pos, a.r) - a.r;
  num = min(num, a.hi);
  uint32_t q = __float2uint_rz(__uint2float_rz(num) * a.rden);
  int32_t rem = static_cast<int32_t>(num - q * a.den);
  const int32_t den = static_cast<int32_t>(a.den);
  const int32_t fix = rem < 0 ? -1 : (rem >= den ? 1 : 0);
  q += static_cast<uint32_t>(fix);
  rem -= fix * den;
  t.i0 = q;
  t.rem = static_cast<uint32_t>(rem);
  t.lam = static_cast<float>(rem) * a.rden;
  t.i1 = min(q + 1, a.in - 1);
  return t;
}

// The tap for any size the interface admits (64-bit numerators).
__device__ __forceinline__ Tap axis_tap_wide(const Axis& a, uint32_t j) {
  Tap t;
  const uint64_t den = 2ull * a.r;
  const uint64_t pos = (2 * (static_cast<uint64_t>(a.origin) + j) + 1) * a.in;  // < 2^46
  uint64_t num = pos > a.r ? pos - a.r : 0;
  const uint64_t hi = static_cast<uint64_t>(a.in - 1) * den;
  num = num < hi ? num : hi;
  const uint64_t q = num / den;
  t.i0 = static_cast<uint32_t>(q);
  t.rem = 0;
  t.lam = static_cast<float>(num - q * den) / static_cast<float>(den);
  t.i1 = t.i0 + 1 < a.in ? t.i0 + 1 : a.in - 1;
  return t;
}

__device__ __forceinline__ Tap axis_tap(const Axis& a, uint32_t j) {
  return a.small ? axis_tap_small(a, j) : axis_tap_wide(a, j);
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

template <int OFF>
__device__ __forceinline__ uint32_t lds32(uint32_t addr) {
  uint32_t v;
  asm volatile("ld.shared.u32 %0, [%1+%2];" : "=r"(v) : "r"(addr), "n"(OFF));
  return v;
}

// ---- arithmetic ---------------------------------------------------------------------------------

// Largest 2 * (resized width) the staged path takes: both weights of a column fit 16 bits
// and 255 * den stays below 2^23, so a weighted sum fits the mantissa of 8388608.0f.
constexpr uint32_t kMaxPackedDen = 32768;

// Horizontal interpolation at shared-memory byte address x (pixel x0, then x0 + 1) as exact
// integers: per channel a * (den - rem) + b * rem, i.e. den times the interpolated value.
// wgt holds (den - rem) in its low half and rem in its high half.  x is unaligned: three
// aligned words are read and shifted; one permute lines up the two taps of two channels for
// a 16-bit-by-8-bit two-way dot product, whose accumulator input 0x4B000000 makes the sum
// the bit pattern of 2^23 + sum; the subtraction that removes 2^23 is exact.
template <int MODE>
__device__ __forceinline__ void hlerp_row(uint32_t x, uint32_t wgt, float n[3]) {
  const uint32_t addr = x & ~3u;
  const uint32_t sh = x << 3;  // the funnel shift takes it modulo 32
  const uint32_t w0 = lds32<0>(addr), w1 = lds32<4>(addr), w2 = lds32<8>(addr);
  const uint32_t lo = __funnelshift_r(w0, w1, sh);  // R0 G0 B0 R1
  const uint32_t hi = __funnelshift_r(w1, w2, sh);  // G1 B1 .. ..
  const uint32_t rg = __byte_perm(lo, hi, 0x4130);  // R0 R1 G0 G1
  const uint32_t bb = __byte_perm(lo, hi, 0x5252);  // B0 B1 B0 B1
  if (MODE == kFloat) {
    n[0] = __uint_as_float(__dp2a_lo(wgt, rg, 0x4B000000u)) - 8388608.0f;
    n[1] = __uint_as_float(__dp2a_hi(wgt, rg, 0x4B000000u)) - 8388608.0f;
    n[2] = __uint_as_float(__dp2a_lo(wgt, bb, 0x4B000000u)) - 8388608.0f;
  } else {  // the rounded modes keep the sums as integers (bit patterns)
    n[0] = __uint_as_float(__dp2a_lo(wgt, rg, 0u));
    n[1] = __uint_as_float(__dp2a_hi(wgt, rg, 0u));
    n[2] = __uint_as_float(__dp2a_lo(wgt, bb, 0u));
  }
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
struct Pack<__nv_bfloat16> {
  using Vec = __nv_bfloat162;
  static __device__ __forceinline__ Vec pair(float x, float y) {
    return __floats2bfloat162_rn(x, y);
  }
  static __device__ __forceinline__ __nv_bfloat16 one(float x) { return __float2bfloat16_rn(x); }
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
  uint32_t wgt[kLaneCols];  // staged path: (den - rem) | rem << 16, the integer weights of the
                            // two taps; direct path: the second tap's weight as float bits
  uint32_t valid;           // bit m: column m exists
};

// Vertical interpolation, normalisation and store of one output row (seven columns).
// q points at this row's column 2 * lane in plane 0.  FULL: every column of every lane
// exists and rows start on even element indices, so pairs go out as one vector each.
template <typename OutT, bool FULL>
__device__ __forceinline__ void emit_row(OutT* __restrict__ q, uint32_t plane, uint32_t lane,
                                         float ly, const float (&hp)[kLaneCols][3],
                                         const float (&hc)[kLaneCols][3], const float (&na)[3],
                                         const float (&nb)[3], uint32_t valid) {
#pragma unroll
  for (int ch = 0; ch < 3; ++ch, q += plane) {
    float o[kLaneCols];
#pragma unroll
    for (int m = 0; m < static_cast<int>(kLaneCols); ++m) {
      const float v = fmaf(ly, hc[m][ch] - hp[m][ch], hp[m][ch]);
      o[m] = fmaf(v, na[ch], nb[ch]);
    }
    OutT* single = q + 192 - lane;  // column 192 + lane
    if (FULL) {
#pragma unroll
      for (int pr = 0; pr < 3; ++pr)
        __stcs(reinterpret_cast<typename Pack<OutT>::Vec*>(q + 64 * pr),
               Pack<OutT>::pair(o[2 * pr], o[2 * pr + 1]));
      __stcs(single, Pack<OutT>::one(o[6]));
    } else {
#pragma unroll
      for (int m = 0; m < 6; ++m)
        if ((valid >> m) & 1u) q[64 * (m >> 1) + (m & 1)] = Pack<OutT>::one(o[m]);
      if ((valid >> 6) & 1u) *single = Pack<OutT>::one(o[6]);
    }
  }
}

// The rounded modes keep den_x times the horizontally interpolated value as a whole number
// (bit pattern of an unsigned integer in the row buffers).  An output pixel is
// floor(num / dd + 1/2) = floor(t / (2 dd)) with t = 2 num + dd, num = prev * (den_y - rem)
// + cur * rem.  The quotient (at most 255) comes from a multiply-high by a reciprocal.
// EXACT (2 dd < 2^22): with 2^k <= 2 dd < 2^(k+1) and magic = ceil(2^(31+k) / (2 dd)),
// floor(t * magic / 2^(31+k)) is the quotient for every t <= 511 dd, because the excess
// t * (magic * 2 dd - 2^(31+k)) stays below 2^(31+k).  Otherwise magic = floor(2^32 / (2 dd)):
// t < 2^32 makes that estimate exact or one short, and the remainder corrects it.
constexpr uint32_t kNoShift = 0xffffffffu;  // Quant::shift when the division needs its correction
struct Quant {
  uint32_t deny2, dd, d2, magic, shift;
};

template <bool EXACT>
__device__ __forceinline__ uint32_t rounded_pixel(float prev, float cur, uint32_t w0, uint32_t w1,
                                                  const Quant& qz) {
  // < 2^32 by the fast path's precondition
  const uint32_t t = __float_as_uint(prev) * w0 + (__float_as_uint(cur) * w1 + qz.dd);
  if (EXACT) return __umulhi(t, qz.magic) >> qz.shift;
  uint32_t q = __umulhi(t, qz.magic);
  if (t - q * qz.d2 >= qz.d2) ++q;
  return q;
}

// Vertical stage of the rounded modes for one output row.  rem is the lower row's integer
// weight (den_y when both taps are the row just staged).  kRoundFloat: q points at column
// 2 * lane of plane 0, as in emit_row.  kU8: q points at the first byte of pixel 2 * lane of
// the output row (HWC); a lane writes its pairs as three 16-bit words each and its single
// column byte by byte.
template <typename OutT, bool FULL, int MODE, bool EXACT>
__device__ __forceinline__ void emit_row_rounded(OutT* __restrict__ q, uint32_t plane,
                                                 uint32_t lane, uint32_t rem,
                                                 const float (&hp)[kLaneCols][3],
                                                 const float (&hc)[kLaneCols][3],
                                                 const Quant& qz, const float (&na)[3],
                                                 const float (&nb)[3], uint32_t valid) {
  const uint32_t w1 = 2 * rem, w0 = qz.deny2 - w1;
  if constexpr (MODE == kU8) {
    uint8_t* b = reinterpret_cast<uint8_t*>(q);
#pragma unroll
    for (int pr = 0; pr < 3; ++pr) {
      uint32_t l[3], r[3];
#pragma unroll
      for (int ch = 0; ch < 3; ++ch) {
        l[ch] = rounded_pixel<EXACT>(hp[2 * pr][ch], hc[2 * pr][ch], w0, w1, qz);
        r[ch] = rounded_pixel<EXACT>(hp[2 * pr + 1][ch], hc[2 * pr + 1][ch], w0, w1, qz);
      }
      uint8_t* at = b + 192 * pr;  // 64 pixels further
      if (FULL) {
        uint16_t* h16 = reinterpret_cast<uint16_t*>(at);  // even byte offset: 6 * lane + 192 * pr
        __stcs(h16, static_cast<uint16_t>(l[0] | (l[1] << 8)));
        __stcs(h16 + 1, static_cast<uint16_t>(l[2] | (r[0] << 8)));
        __stcs(h16 + 2, static_cast<uint16_t>(r[1] | (r[2] << 8)));
      } else {
#pragma unroll
        for (int ch = 0; ch < 3; ++ch) {
          if ((valid >> (2 * pr)) & 1u) at[ch] = static_cast<uint8_t>(l[ch]);
          if ((valid >> (2 * pr + 1)) & 1u) at[3 + ch] = static_cast<uint8_t>(r[ch]);
        }
      }
    }
    uint8_t* single = b + 3 * (192 - lane);  // pixel 192 + lane
    if (FULL || ((valid >> 6) & 1u)) {
#pragma unroll
      for (int ch = 0; ch < 3; ++ch)
        single[ch] = static_cast<uint8_t>(rounded_pixel<EXACT>(hp[6][ch], hc[6][ch], w0, w1, qz));
    }
  } else {
#pragma unroll
    for (int ch = 0; ch < 3; ++ch, q += plane) {
      float o[kLaneCols];
#pragma unroll
      for (int m = 0; m < static_cast<int>(kLaneCols); ++m) {
        const uint32_t px = rounded_pixel<EXACT>(hp[m][ch], hc[m][ch], w0, w1, qz);
        o[m] = fmaf(__uint_as_float(0x4B000000u | px) - 8388608.0f, na[ch], nb[ch]);
      }
      OutT* single = q + 192 - lane;
      if (FULL) {
#pragma unroll
        for (int pr = 0; pr < 3; ++pr)
          __stcs(reinterpret_cast<typename Pack<OutT>::Vec*>(q + 64 * pr),
                 Pack<OutT>::pair(o[2 * pr], o[2 * pr + 1]));
        __stcs(single, Pack<OutT>::one(o[6]));
      } else {
#pragma unroll
        for (int m = 0; m < 6; ++m)
          if ((valid >> m) & 1u) q[64 * (m >> 1) + (m & 1)] = Pack<OutT>::one(o[m]);
        if ((valid >> 6) & 1u) *single = Pack<OutT>::one(o[6]);
      }
    }
  }
}

// One axis in 64-bit integers: tap, clamped neighbour, remainder and denominator (the direct
// path of the rounded modes, any size the interface admits).
struct TapInt {
  uint32_t i0, i1;
  uint64_t rem, den;
};

__device__ __forceinline__ TapInt axis_tap_int(uint32_t in, uint32_t r, uint32_t origin,
                                               uint32_t j) {
  TapInt t;
  t.den = 2ull * r;
  const uint64_t pos = (2 * (static_cast<uint64_t>(origin) + j) + 1) * in;
  uint64_t num = pos > r ? pos - r : 0;
  const uint64_t hi = static_cast<uint64_t>(in - 1) * t.den;
  num = num < hi ? num : hi;
  const uint64_t q = num / t.den;
  t.i0 = static_cast<uint32_t>(q);
  t.i1 = t.i0 + 1 < in ? t.i0 + 1 : in - 1;
  t.rem = num - q * t.den;
  return t;
}

// The rounded pixel from its four taps, exact at any size (products pass 2^64).
__device__ __forceinline__ uint32_t rounded_pixel_wide(uint32_t p00, uint32_t p01, uint32_t p10,
                                                       uint32_t p11, const TapInt& tx,
                                                       const TapInt& ty) {
  typedef unsigned __int128 u128;
  const u128 upper = static_cast<u128>(p00) * (tx.den - tx.rem) + static_cast<u128>(p01) * tx.rem;
  const u128 lower = static_cast<u128>(p10) * (tx.den - tx.rem) + static_cast<u128>(p11) * tx.rem;
  const u128 num = upper * (ty.den - ty.rem) + lower * ty.rem;
  const u128 den = static_cast<u128>(tx.den) * ty.den;
  // the quotient is at most 255: find it by comparison instead of a 128-bit division
  const u128 t = 2 * num + den, d2 = 2 * den;
  uint32_t q = 0;
#pragma unroll 1
  for (int bit = 7; bit >= 0; --bit) {
    const uint32_t trial = q | (1u << bit);
    if (static_cast<u128>(trial) * d2 <= t) q = trial;
  }
  return q;
}

// ---- task preparation: geometry of a slab into the warp's meta buffer --------------------------

struct Issue {          // the copy stream's view of the task it is issuing
  const uint8_t* base;  // image base + 3 * xmin
  uint32_t pitch;       // 3 * w
  uint32_t copy_bytes;  // tapped bytes of a row
  uint32_t stride;
  uint32_t rpg;         // rows per group
  uint32_t n_list;
  uint32_t buf;         // meta buffer of the task
};

// Fills `m` for task `task`; returns its kind.  All lanes take part.
template <int MODE, bool CROP>
__device__ __forceinline__ uint32_t prepare(const Params& p, uint32_t task, TaskMeta& m,
                                            uint32_t lane, Issue& is) {
  const uint32_t C = p.C;
  const uint32_t per_img = p.slabs * p.col_blocks;
  const uint32_t img = task / per_img;
  const uint32_t rest = task - img * per_img;
  const uint32_t slab = rest / p.col_blocks;
  const uint32_t cb = rest - slab * p.col_blocks;
  const preba_img_t e = p.table[img];
  uint32_t kind = kSkip;
  if (entry_ok(e, p.pixels_bytes)) {
    // S <= 2^14 and sides <= 2^15: the product fits 32 bits
    const uint32_t lng = max(e.h, e.w), sht = min(e.h, e.w);
    const uint32_t rl = p.S * lng / sht;
    const uint32_t rh = e.h <= e.w ? p.S : rl;
    const uint32_t rw = e.h <= e.w ? rl : p.S;
    uint32_t top = (rh - C) / 2, left = (rw - C) / 2;  // rh, rw >= S >= C
    bool window_ok = true;
    if (CROP) {
      const uint32_t t = p.crop[2 * img], l = p.crop[2 * img + 1];
      window_ok = t <= rh - C && l <= rw - C;
      top = min(t, rh - C);  // a window that does not fit is reported and skipped below
      left = min(l, rw - C);
    }
    const uint32_t k0 = slab * p.slab_rows;
    const uint32_t rows_out = min(p.slab_rows, C - k0);
    const uint32_t col0 = cb * kTaskCols;
    const uint32_t cols = min(kTaskCols, C - col0);
    const Axis ax = make_axis(e.w, rw, left, C);
    const Axis ay = make_axis(e.h, rh, top, C);
    const bool active = lane < rows_out;
    Tap tf, tl, ty;
    if (ax.small && ay.small) {
      tf = axis_tap_small(ax, col0);
      tl = axis_tap_small(ax, col0 + cols - 1);
      ty = axis_tap_small(ay, k0 + (active ? lane : 0u));
    } else {
      tf = axis_tap(ax, col0);
      tl = axis_tap(ax, col0 + cols - 1);
      ty = axis_tap(ay, k0 + (active ? lane : 0u));
    }
    const uint32_t xmin = tf.i0;
    const uint32_t copy_px = tl.i1 - xmin + 1;
    // a lane reads 12 bytes from the word holding its first tap, which may be the last
    // staged pixel: leave room for one more pixel and the word overshoot
    const uint32_t stride = (15 + 3 * copy_px + 3 + 12 + 15) & ~15u;
    const uint32_t rpg = min(kGroupRows, kGroupBytes / stride);
    const uint64_t end16 = (e.offset + 3ull * e.h * e.w + 15) & ~15ull;
    kind = (rpg >= 1 && end16 <= p.pixels_bytes && ax.small && ax.den <= kMaxPackedDen)
               ? kStream : kGather;
    // rounded modes: 32-bit arithmetic needs 2 * num + dd <= 511 * dd below 2^32
    const uint64_t dd = static_cast<uint64_t>(ax.den) * ay.den;
    if (MODE != kFloat && !(ay.small && 511ull * dd < (1ull << 32))) kind = kGather;
    if (!window_ok) kind = kSkip;

    // rows of the slab: the ascending list of distinct source rows.  Output row `lane`
    // lists its lower tap if that lies beyond the previous row's upper tap, and its upper
    // tap if that is a new row too.
    const uint32_t y1_prev = __shfl_up_sync(0xffffffffu, ty.i1, 1);
    const bool new0 = active && (lane == 0 || ty.i0 > y1_prev);
    const bool new1 = active && ty.i1 != ty.i0 && (lane == 0 || ty.i1 > y1_prev);
    const uint32_t b0 = __ballot_sync(0xffffffffu, new0);
    const uint32_t b1 = __ballot_sync(0xffffffffu, new1);
    const uint32_t below = (1u << lane) - 1u;
    const uint32_t excl = static_cast<uint32_t>(__popc(b0 & below) + __popc(b1 & below));
    const uint32_t n_list = static_cast<uint32_t>(__popc(b0) + __popc(b1));
    // The last row a lane lists completes this output row and those after it up to the
    // next lane that lists a row.
    const uint32_t above = (b0 | b1) & ~((2u << lane) - 1u);
    const uint32_t done = (above ? static_cast<uint32_t>(__ffs(above) - 1) : rows_out) - lane;
    if (new0) {
      m.row[excl] = ty.i0;
      m.info[excl] = ((new1 ? 0u : done) << 8) | ((3u * (ty.i0 * e.w + xmin)) & 15u);
    }
    if (new1) {
      const uint32_t at = excl + (new0 ? 1u : 0u);
      m.row[at] = ty.i1;
      m.info[at] = (done << 8) | ((3u * (ty.i1 * e.w + xmin)) & 15u);
    }
    if (MODE == kFloat) {
      if (active) m.lam[lane] = __float_as_uint(ty.i1 == ty.i0 ? 1.0f : ty.lam);
    } else {
      // integer weight of the lower row; all of it when both taps are the row just staged
      if (active) m.lam[lane] = ty.i1 == ty.i0 ? ay.den : ty.rem;
      if (lane == 0 && kind == kStream) {
        m.deny2 = 2 * ay.den;
        m.dd = static_cast<uint32_t>(dd);
        const uint64_t d2 = 2 * dd;  // >= 8
        if (d2 < (1ull << 22)) {
          const uint32_t k = 31 - static_cast<uint32_t>(__clz(static_cast<uint32_t>(d2)));
          m.magic = static_cast<uint32_t>(((1ull << (31 + k)) + d2 - 1) / d2);
          m.shift = k - 1;
        } else {
          m.magic = static_cast<uint32_t>((1ull << 32) / d2);
          m.shift = kNoShift;
        }
      }
    }
    if (lane == 0) {
      m.top = top;
      m.left = left;
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
      m.src = e.offset;
    }
    is.base = p.pixels + e.offset + 3 * xmin;
    is.pitch = 3 * e.w;
    is.copy_bytes = 3 * copy_px;
    is.stride = stride;
    is.rpg = rpg;
    is.n_list = kind == kStream ? n_list : 0;
    if (!window_ok && lane == 0) report(p.status, PREBA_ERR_BAD_CROP);
  } else {
    if (lane == 0) report(p.status, PREBA_ERR_BAD_TABLE);
    is.n_list = 0;
  }
  if (lane == 0) m.kind = kind;
  __syncwarp();
  return kind;
}

// Direct path of the rounded modes for one task: exact integers of any size, taps from
// global memory.
template <typename OutT, int MODE>
__device__ __forceinline__ void gather_rounded(const Params& p, const TaskMeta& cm, uint32_t lane) {
  const uint32_t C = p.C;
  const size_t plane = static_cast<size_t>(C) * C;
  const uint32_t w = cm.w, h = cm.h, rw = cm.rw, rh = cm.rh, col0 = cm.col0;
  const uint8_t* __restrict__ src = p.pixels + cm.src;
  const size_t pitch = 3 * static_cast<size_t>(w);
  for (uint32_t t = 0; t < cm.rows_out; ++t) {
    const TapInt ty = axis_tap_int(h, rh, cm.top, cm.k0 + t);
    const uint8_t* r0 = src + ty.i0 * pitch;
    const uint8_t* r1 = src + ty.i1 * pitch;
#pragma unroll 1
    for (int m = 0; m < static_cast<int>(kLaneCols); ++m) {
      const uint32_t j = col0 + lane_col(lane, m);
      if (j >= C) continue;
      const TapInt tx = axis_tap_int(w, rw, cm.left, j);
#pragma unroll 1
      for (uint32_t ch = 0; ch < 3; ++ch) {
        const uint32_t v = rounded_pixel_wide(__ldg(r0 + 3 * static_cast<size_t>(tx.i0) + ch),
                                              __ldg(r0 + 3 * static_cast<size_t>(tx.i1) + ch),
                                              __ldg(r1 + 3 * static_cast<size_t>(tx.i0) + ch),
                                              __ldg(r1 + 3 * static_cast<size_t>(tx.i1) + ch), tx, ty);
        const size_t row = static_cast<size_t>(cm.k0 + t) * C + j;
        if constexpr (MODE == kU8) {
          reinterpret_cast<uint8_t*>(p.out)[3 * (static_cast<size_t>(cm.img) * plane + row) + ch] =
              static_cast<uint8_t>(v);
        } else {
          const float o = fmaf(static_cast<float>(v), p.a[ch], p.b[ch]);
          static_cast<OutT*>(p.out)[(static_cast<size_t>(cm.img) * 3 + ch) * plane + row] =
              Pack<OutT>::one(o);
        }
      }
    }
  }
}

template <typename OutT, bool FULL, int MODE>
__device__ __forceinline__ void emit_any(OutT* __restrict__ q, uint32_t plane, uint32_t lane,
                                         uint32_t weight_bits,
                                         const float (&prev)[kLaneCols][3],
                                         const float (&cur)[kLaneCols][3], const float (&sa)[3],
                                         const float (&nb)[3], const Quant& qz, uint32_t valid) {
  if constexpr (MODE == kFloat)
    emit_row<OutT, FULL>(q, plane, lane, __uint_as_float(weight_bits), prev, cur, sa, nb, valid);
  else if (qz.shift != kNoShift)
    emit_row_rounded<OutT, FULL, MODE, true>(q, plane, lane, weight_bits, prev, cur, qz, sa, nb,
                                             valid);
  else
    emit_row_rounded<OutT, FULL, MODE, false>(q, plane, lane, weight_bits, prev, cur, qz, sa, nb,
                                              valid);
}

// ---- the warp program ---------------------------------------------------------------------------------

template <typename OutT, int MODE, bool CROP>
__device__ __forceinline__ void warp_main(const Params& p, WarpShared& ws, uint32_t lane,
                                          uint32_t gwarp, uint32_t nwarps) {
  const uint32_t C = p.C;
  const uint32_t plane = C * C;
  const uint32_t row_step = MODE == kU8 ? 3 * C : C;  // elements of OutT between output rows
  const float nb[3] = {p.b[0], p.b[1], p.b[2]};
  float sa[3] = {0.f, 0.f, 0.f};  // staged path: 1 / (255 * std * den) of the task's image
  Quant qz = {0, 0, 0, 0, 0};     // rounded modes: the task's division constants

  // task claims: a warp's first task is its own index; later ones come from the shared
  // counter (dynamic) or every nwarps-th task (static)
  uint32_t next_task = gwarp;
  uint32_t turn = 0;

  // copy stream
  Issue is;
  is.base = p.pixels;
  is.pitch = is.copy_bytes = is.stride = 0;
  is.n_list = 0;
  is.rpg = 1;
  is.buf = 0;
  uint32_t is_row = 0;       // next listed row of the issuing task to copy
  uint32_t prepared = 0;     // tasks prepared (meta buffers written)
  uint32_t issued = 0;       // groups issued
  bool ended = false;        // no task left to prepare

  // compute stream
  uint32_t finished = 0;     // tasks computed
  uint32_t consumed = 0;     // groups computed
  bool need_task = true;
  bool failed = false;
  Lane ln;
  float hA[kLaneCols][3], hB[kLaneCols][3];
  uint32_t par = 0;          // which of hA/hB receives the next row
  uint32_t c_row = 0, c_nlist = 0, c_rpg = 1, c_stride = 0, t_out = 0;
  bool full = false;
  const TaskMeta* cm = &ws.meta[0];
  OutT* q_out = static_cast<OutT*>(p.out);  // column 2 * lane of the next output row, plane 0
#pragma unroll
  for (int m = 0; m < static_cast<int>(kLaneCols); ++m) {
    ln.off[m] = 0;
    ln.wgt[m] = 0;
#pragma unroll
    for (int ch = 0; ch < 3; ++ch) hA[m][ch] = hB[m][ch] = 0.f;
  }
  ln.valid = 0;

  for (;;) {
    // -- advance the copy stream: at most kGroups groups and kMetaBufs - 1 tasks ahead -------
    for (;;) {
      if (is_row < is.n_list) {
        if (issued >= consumed + kGroups) break;
        const uint32_t slot = issued % kGroups;
        const uint32_t cnt = min(is.rpg, is.n_list - is_row);
        const uint32_t bar = smem_addr(&ws.full[slot]);
        if (lane < kGroupRows) {
          if (lane < cnt) {
            const uint8_t* src = is.base +
                static_cast<size_t>(ws.meta[is.buf].row[is_row + lane]) * is.pitch;
            const uintptr_t s = reinterpret_cast<uintptr_t>(src);
            const uintptr_t s0 = s & ~static_cast<uintptr_t>(15);
            const uint32_t bytes = static_cast<uint32_t>(
                ((s + is.copy_bytes + 15) & ~static_cast<uintptr_t>(15)) - s0);
            fence_async_shared();
            // checked build: the row lies in its ring group and in the pixel buffer
            if (PREBA_IN_RANGE(p.status,
                               lane * is.stride + bytes <= kGroupBytes &&
                                   s0 >= reinterpret_cast<uintptr_t>(p.pixels) &&
                                   s0 - reinterpret_cast<uintptr_t>(p.pixels) + bytes <=
                                       p.pixels_bytes)) {
              mbar_arrive_expect_tx(bar, bytes);
              bulk_copy_g2s(smem_addr(&ws.ring[slot][lane * is.stride]),
                            reinterpret_cast<const void*>(s0), bytes, bar);
            } else {
              mbar_arrive(bar);
            }
          } else {
            mbar_arrive(bar);
          }
        }
        is_row += cnt;
        ++issued;
      } else {
        if (ended || prepared - finished >= kMetaBufs) break;
        // the claim made while the previous task was prepared has arrived by now
        const uint32_t task = p.sched ? __shfl_sync(0xffffffffu, next_task, 0) : next_task;
        if (p.sched) {
          if (lane == 0) next_task = nwarps + atomicAdd(&p.sched[0], 1u);
        } else {
          ++turn;
          const uint64_t t = static_cast<uint64_t>(gwarp) + static_cast<uint64_t>(turn) * nwarps;
          next_task = t < p.tasks ? static_cast<uint32_t>(t) : p.tasks;
        }
        const uint32_t buf = prepared % kMetaBufs;
        if (task >= p.tasks) {
          if (lane == 0) ws.meta[buf].kind = kEnd;
          __syncwarp();
          ended = true;
          is.n_list = 0;
        } else {
          (void)prepare<MODE, CROP>(p, task, ws.meta[buf], lane, is);
        }
        is.buf = buf;
        is_row = 0;
        ++prepared;
      }
    }

    // -- compute stream: start the next task, or one group of the current one ------------------
    if (need_task) {
      if (finished == prepared) break;
      cm = &ws.meta[finished % kMetaBufs];
      const uint32_t kind = cm->kind;
      if (kind == kEnd) break;
      if (kind == kSkip) {
        ++finished;
        continue;
      }
      const uint32_t w = cm->w, rw = cm->rw, col0 = cm->col0, xmin = cm->xmin;
      const Axis ax = make_axis(w, rw, CROP ? cm->left : (rw - C) / 2, C);
      ln.valid = 0;
      if (kind == kStream) {  // implies ax.small and den <= kMaxPackedDen
#pragma unroll
        for (int m = 0; m < static_cast<int>(kLaneCols); ++m) {
          const uint32_t j = col0 + lane_col(lane, m);
          if (j < C) ln.valid |= 1u << m;
          const Tap t = axis_tap_small(ax, min(j, C - 1));
          ln.off[m] = 3 * (t.i0 - xmin);
          ln.wgt[m] = (ax.den - t.rem) | (t.rem << 16);
        }
        if (MODE == kFloat) {
          // staged rows carry den times the pixel value: fold 1 / den into the scale
#pragma unroll
          for (int ch = 0; ch < 3; ++ch) sa[ch] = p.a[ch] * ax.rden;
        } else {
          qz.deny2 = cm->deny2;
          qz.dd = cm->dd;
          qz.d2 = 2 * qz.dd;
          qz.magic = cm->magic;
          qz.shift = cm->shift;
#pragma unroll
          for (int ch = 0; ch < 3; ++ch) sa[ch] = p.a[ch];
        }
      } else {
#pragma unroll
        for (int m = 0; m < static_cast<int>(kLaneCols); ++m) {
          const uint32_t j = col0 + lane_col(lane, m);
          if (j < C) ln.valid |= 1u << m;
          const Tap t = axis_tap(ax, min(j, C - 1));
          ln.off[m] = 3 * (t.i0 - xmin);
          ln.wgt[m] = __float_as_uint(t.lam);
        }
      }
      full = (C & 1u) == 0 && __all_sync(0xffffffffu, ln.valid == 0x7fu);
      if (MODE == kU8)  // HWC: first byte of pixel col0 + 2 * lane in row k0
        q_out = static_cast<OutT*>(p.out) +
                3 * (static_cast<size_t>(cm->img) * plane + (cm->k0 * C + col0 + 2 * lane));
      else
        q_out = static_cast<OutT*>(p.out) + static_cast<size_t>(cm->img) * 3 * plane +
                (cm->k0 * C + col0 + 2 * lane);
      c_nlist = cm->n_list;
      c_rpg = cm->rows_per_group;
      c_stride = cm->stride;
      c_row = 0;
      t_out = 0;
      need_task = false;
      if (kind != kGather) {
        // staged: the groups follow
      } else if constexpr (MODE != kFloat) {
        gather_rounded<OutT, MODE>(p, *cm, lane);
        ++finished;
        need_task = true;
      } else {
        // direct path: taps straight from global memory (footprint too wide for the ring)
        const uint8_t* __restrict__ src = p.pixels + cm->src + 3 * xmin;
        const size_t pitch = 3 * static_cast<size_t>(w);
        const uint32_t h = cm->h, rh = cm->rh;
        const Axis ay = make_axis(h, rh, CROP ? cm->top : (rh - C) / 2, C);
        const float na[3] = {p.a[0], p.a[1], p.a[2]};
        for (uint32_t t = 0; t < cm->rows_out; ++t, q_out += row_step) {
          const Tap ty = axis_tap(ay, cm->k0 + t);
          const uint8_t* r0 = src + ty.i0 * pitch;
          const uint8_t* r1 = src + ty.i1 * pitch;
#ifdef PREBA_CHECKED
          {  // both rows and every tap of the lane inside the image, the output row inside the crop
            bool fits = ty.i0 < h && ty.i1 < h && cm->k0 + t < C && cm->img < p.n &&
                        cm->src + 3ull * h * w <= p.pixels_bytes;
#pragma unroll
            for (int m = 0; m < static_cast<int>(kLaneCols); ++m)
              fits = fits && 3 * xmin + ln.off[m] + 6 <= 3 * w + (ln.wgt[m] ? 0u : 3u);
            if (!PREBA_IN_RANGE(p.status, __all_sync(0xffffffffu, fits))) continue;
          }
#endif
#pragma unroll
          for (int m = 0; m < static_cast<int>(kLaneCols); ++m) {
            // the right neighbour is read only where it carries weight (it exists then)
            const float lam = __uint_as_float(ln.wgt[m]);
            const uint32_t nbr = lam > 0.f ? 3u : 0u;
#pragma unroll
            for (int ch = 0; ch < 3; ++ch) {
              float a = __ldg(r0 + ln.off[m] + ch), b = __ldg(r0 + ln.off[m] + nbr + ch);
              hA[m][ch] = fmaf(lam, b - a, a);
              a = __ldg(r1 + ln.off[m] + ch), b = __ldg(r1 + ln.off[m] + nbr + ch);
              hB[m][ch] = fmaf(lam, b - a, a);
            }
          }
          emit_row<OutT, false>(q_out, plane, lane, ty.lam, hA, hB, na, nb, ln.valid);
        }
        // the staged path relies on whole numbers in the row buffers
#pragma unroll
        for (int m = 0; m < static_cast<int>(kLaneCols); ++m)
#pragma unroll
          for (int ch = 0; ch < 3; ++ch) hA[m][ch] = hB[m][ch] = 0.f;
        ++finished;
        need_task = true;
      }
      continue;
    }

    // one group of staged rows
    {
      const uint32_t slot = consumed % kGroups;
      if (!mbar_wait(smem_addr(&ws.full[slot]), (consumed / kGroups) & 1)) {
        failed = true;
        break;
      }
      const uint32_t cnt = min(c_rpg, c_nlist - c_row);
      uint32_t row_addr = smem_addr(&ws.ring[slot][0]);
      for (uint32_t r = 0; r < cnt; ++r, row_addr += c_stride) {
#ifdef PREBA_CHECKED
        // every index and offset of this row before it is used: the list entry, the 12 bytes
        // each column reads from the ring group, the output rows the row completes
        bool fits = c_row + r < kMaxList;
        if (fits) {
          const uint32_t info_c = cm->info[c_row + r];
          const uint32_t lo = smem_addr(&ws.ring[slot][0]), hi = lo + kGroupBytes;
          const uint32_t base_c = row_addr + (info_c & 0xffu);
#pragma unroll
          for (int m = 0; m < static_cast<int>(kLaneCols); ++m) {
            const uint32_t at = (base_c + ln.off[m]) & ~3u;
            fits = fits && at >= lo && at + 12 <= hi;
          }
          fits = fits && t_out + (info_c >> 8) <= 32 && cm->k0 + t_out + (info_c >> 8) <= C &&
                 cm->img < p.n;
        }
        if (!PREBA_IN_RANGE(p.status, __all_sync(0xffffffffu, fits))) {
          par ^= 1u;
          continue;
        }
#endif
        const uint32_t info = cm->info[c_row + r];
        const uint32_t base = row_addr + (info & 0xffu);  // the row's first tapped byte
        uint32_t e = info >> 8;
        if (par == 0) {
#pragma unroll
          for (int m = 0; m < static_cast<int>(kLaneCols); ++m)
            hlerp_row<MODE>(base + ln.off[m], ln.wgt[m], hA[m]);
#pragma unroll 1
          for (; e > 0; --e, ++t_out, q_out += row_step) {
            const uint32_t wy = cm->lam[t_out];
            if (full)
              emit_any<OutT, true, MODE>(q_out, plane, lane, wy, hB, hA, sa, nb, qz, ln.valid);
            else
              emit_any<OutT, false, MODE>(q_out, plane, lane, wy, hB, hA, sa, nb, qz, ln.valid);
          }
        } else {
#pragma unroll
          for (int m = 0; m < static_cast<int>(kLaneCols); ++m)
            hlerp_row<MODE>(base + ln.off[m], ln.wgt[m], hB[m]);
#pragma unroll 1
          for (; e > 0; --e, ++t_out, q_out += row_step) {
            const uint32_t wy = cm->lam[t_out];
            if (full)
              emit_any<OutT, true, MODE>(q_out, plane, lane, wy, hA, hB, sa, nb, qz, ln.valid);
            else
              emit_any<OutT, false, MODE>(q_out, plane, lane, wy, hA, hB, sa, nb, qz, ln.valid);
          }
        }
        par ^= 1u;
      }
      c_row += cnt;
      ++consumed;
      __syncwarp();  // every lane is done with the slot before the stream refills it
      if (c_row >= c_nlist) {
        ++finished;
        need_task = true;
      }
    }
  }

  if (failed) {
    if (lane == 0) report(p.status, PREBA_ERR_TIMEOUT);
    // copies already issued may still be landing in this warp's ring: wait for them
    // (bounded) before the CTA can retire
    for (uint32_t q = consumed; q < issued; ++q)
      (void)mbar_wait(smem_addr(&ws.full[q % kGroups]), (q / kGroups) & 1);
  }
  // A launch marked as overlapping started without waiting for the kernels before it on the
  // stream.  It must not complete before them, or work ordered after it could run ahead of
  // their results: wait here, after the last store, until they have completed (no wait at all
  // for an unmarked launch).  Each launch waits for its predecessor, so completion follows
  // the stream's order along a whole chain of marked launches.
  asm volatile("griddepcontrol.wait;" ::: "memory");
  // the last warp out leaves the claim counters at zero for the next launch
  if (p.sched && lane == 0) {
    __threadfence();
    if (atomicAdd(&p.sched[1], 1u) == nwarps - 1) {
      p.sched[0] = 0;
      p.sched[1] = 0;
    }
  }
}

// The rounded modes keep integer row state and division constants on top of what the float
// mode holds: at four CTAs per SM (128 registers) they spill, so they run three per SM.
#ifdef PREBA_CHECKED
#define PREBA_FUSED_CTAS(MODE) ((void)kCtasPerSm, 2)  // the range checks cost registers
#else
#define PREBA_FUSED_CTAS(MODE) ((MODE) == kFloat ? kCtasPerSm : kCtasPerSm - 1)
#endif
template <typename OutT, int MODE, bool CROP>
__global__ void __launch_bounds__(kThreads, PREBA_FUSED_CTAS(MODE))
    preba_fused_kernel(const Params p) {
  __shared__ WarpShared sm[kWarpsPerCta];
  // a following launch that was marked independent of this one may start as soon as
  // resources free up
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const uint32_t lane = threadIdx.x & 31;
  // read through a shuffle so that the compiler treats the warp's index, and the shared-memory
  // addresses derived from it, as the same in every lane
  const uint32_t warp = __shfl_sync(0xffffffffu, threadIdx.x >> 5, 0);
  WarpShared& ws = sm[warp];
  if (lane == 0) {
    for (uint32_t g = 0; g < kGroups; ++g) mbar_init(smem_addr(&ws.full[g]), kGroupRows);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncwarp();
  warp_main<OutT, MODE, CROP>(p, ws, lane, blockIdx.x * kWarpsPerCta + warp, gridDim.x * kWarpsPerCta);
}

thread_local int g_last_cuda_error = 0;

int check_args(const uint8_t* pixels, uint64_t pixels_bytes, const void* table, uint32_t n,
               const void* out, uint64_t out_bytes, uint32_t out_size, uint32_t resize_short,
               const float mean[3], const float std[3], int out_dtype, bool allow_u8 = false) {
  if (!pixels || !table || !out || !mean || !std || n == 0) return PREBA_ERR_INVALID_ARG;
  if (!(dtype_ok(out_dtype) || (allow_u8 && out_dtype == PREBA_U8)) || out_size == 0 || resize_short < out_size ||
      resize_short > PREBA_MAX_RESIZE)
    return PREBA_ERR_INVALID_ARG;
  for (int c = 0; c < 3; ++c)
    if (!std::isfinite(mean[c]) || !std::isfinite(std[c]) || std[c] == 0.0f)
      return PREBA_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(pixels) % 16 || reinterpret_cast<uintptr_t>(out) % 16 ||
      reinterpret_cast<uintptr_t>(table) % 8)
    return PREBA_ERR_INVALID_ARG;
  const uint64_t need = static_cast<uint64_t>(n) * 3ull * out_size * out_size *
                        dtype_bytes(out_dtype);
  if (out_bytes < need) return PREBA_ERR_BUFFER_TOO_SMALL;
  if (pixels_bytes == 0) return PREBA_ERR_BUFFER_TOO_SMALL;
  const uint64_t tasks = static_cast<uint64_t>(n) * ((out_size + kMinSlabRows - 1) / kMinSlabRows) *
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

// The kernel for an output type and mode.
using KernelFn = void (*)(const Params);
constexpr int kVariants = 14;

// 0..2: fp32/fp16/bf16 out; 3..5: the same after rounding; 6: uint8 out; +7: with a crop
// window per image (Params::crop).
int variant_of(int out_dtype, int mode, bool crop) {
  const int t = out_dtype == PREBA_F16 ? 1 : out_dtype == PREBA_BF16 ? 2 : 0;
  const int base = mode == kU8 ? 6 : (mode == kRoundFloat ? 3 : 0) + t;
  return base + (crop ? 7 : 0);
}

template <bool CROP>
KernelFn kernel_with(int base) {
  switch (base) {
    case 1: return preba_fused_kernel<__half, kFloat, CROP>;
    case 2: return preba_fused_kernel<__nv_bfloat16, kFloat, CROP>;
    case 3: return preba_fused_kernel<float, kRoundFloat, CROP>;
    case 4: return preba_fused_kernel<__half, kRoundFloat, CROP>;
    case 5: return preba_fused_kernel<__nv_bfloat16, kRoundFloat, CROP>;
    case 6: return preba_fused_kernel<uint8_t, kU8, CROP>;
    default: return preba_fused_kernel<float, kFloat, CROP>;
  }
}

KernelFn kernel_of(int variant) {
  return variant >= 7 ? kernel_with<true>(variant - 7) : kernel_with<false>(variant);
}

// Resident CTAs of the fused kernel on the current device (grid of a persistent launch).
// The answer depends on the device and the kernel only; it is computed once per device and
// kernel variant and kept (a benign race: concurrent first calls store the same value).
int resident_ctas(int variant, cudaError_t* err) {
  constexpr int kMaxDevices = 64;
  static std::atomic<int> cache[kVariants][kMaxDevices];
  int dev = 0;
  *err = cudaGetDevice(&dev);
  if (*err != cudaSuccess) return 0;
  if (dev >= 0 && dev < kMaxDevices) {
    const int known = cache[variant][dev].load(std::memory_order_relaxed);
    if (known > 0) return known;
  }
  int sms = 0, per_sm = 0;
  *err = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (*err != cudaSuccess) return 0;
  *err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel_of(variant), kThreads, 0);
  if (*err != cudaSuccess) return 0;
  const int resident = sms * (per_sm > 0 ? per_sm : 1);
  if (dev >= 0 && dev < kMaxDevices)
    cache[variant][dev].store(resident, std::memory_order_relaxed);
  return resident;
}

int launch(const Params& given, int out_dtype, bool overlap, cudaStream_t stream,
           int mode = kFloat) {
  cudaError_t err = cudaSuccess;
  const int variant = variant_of(out_dtype, mode, given.crop != nullptr);
  const int resident = resident_ctas(variant, &err);
  Params p = given;
  if (err == cudaSuccess && !overlap) {
    // A launch that runs alone is as long as the work of its busiest warp: the rounds of tasks
    // the resident warps need, times a task's rows (plus about four rows' worth of set-up and
    // halo per task).  The slab height that makes this smallest is taken, between the full 32
    // rows and kMinSlabRows (ties: the taller slab): 256 images of 224 rows get nine slabs of
    // 25 rows each, one per warp, instead of fourteen of 16.  The arithmetic per output
    // element, and so the result, does not depend on the split.  Launches marked as
    // overlapping their predecessor keep 32-row slabs: there the GPU is kept busy by the
    // neighbouring launches and throughput counts.
    const uint64_t warps = static_cast<uint64_t>(resident) * kWarpsPerCta;
    uint64_t best_cost = ~0ull;
    uint32_t best_rows = p.slab_rows;
    for (uint32_t r = p.slab_rows; r >= kMinSlabRows; --r) {
      const uint64_t tasks = static_cast<uint64_t>(p.n) * ((p.C + r - 1) / r) * p.col_blocks;
      const uint64_t cost = ((tasks + warps - 1) / warps) * (r + 4u);
      if (cost < best_cost) best_cost = cost, best_rows = r;
      if (r == 1) break;
    }
    p.slab_rows = best_rows;
    p.slabs = (p.C + p.slab_rows - 1) / p.slab_rows;
    p.tasks = static_cast<uint32_t>(static_cast<uint64_t>(p.n) * p.slabs * p.col_blocks);
  }
  if (err == cudaSuccess) {
    const uint32_t want = (p.tasks + kWarpsPerCta - 1) / kWarpsPerCta;
    const uint32_t blocks = want < static_cast<uint32_t>(resident) ? want : resident;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(blocks);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = overlap ? 1 : 0;
    err = cudaLaunchKernelEx(&cfg, kernel_of(variant), p);
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
  p.crop = nullptr;
  p.col_blocks = (out_size + kTaskCols - 1) / kTaskCols;
  p.slab_rows = kSlabRows;
  p.slabs = (out_size + p.slab_rows - 1) / p.slab_rows;
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
  if (batch->flags & ~PREBA_OVERLAP_PREVIOUS) return PREBA_ERR_INVALID_ARG;
  if (batch->table_host) {
    rc = check_table(batch->table_host, batch->n, batch->pixels_bytes);
    if (rc != PREBA_OK) return rc;
  }
  const Params p = make_params(batch->pixels, batch->pixels_bytes, batch->table, batch->n,
                               batch->out, batch->status, batch->scratch, out_size, resize_short,
                               mean, std);
  return launch(p, out_dtype, (batch->flags & PREBA_OVERLAP_PREVIOUS) != 0,
                static_cast<cudaStream_t>(stream));
}

extern "C" int preba_preprocess_ex(const preba_batch_t* batch, const preba_options_t* opt,
                                   void* stream) {
  using namespace preba;
  if (!batch || !opt) return PREBA_ERR_INVALID_ARG;
  if (opt->flags & ~PREBA_EX_ROUND_U8) return PREBA_ERR_INVALID_ARG;
  const bool round_u8 = (opt->flags & PREBA_EX_ROUND_U8) != 0;
  if (opt->out_dtype == PREBA_U8 && !round_u8) return PREBA_ERR_INVALID_ARG;
  int rc = check_args(batch->pixels, batch->pixels_bytes, batch->table, batch->n, batch->out,
                      batch->out_bytes, opt->out_size, opt->resize_short, opt->mean, opt->std,
                      opt->out_dtype, true);
  if (rc != PREBA_OK) return rc;
  if (reinterpret_cast<uintptr_t>(batch->scratch) % 16) return PREBA_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(opt->crop_origin) % 4) return PREBA_ERR_INVALID_ARG;
  if (batch->flags & ~PREBA_OVERLAP_PREVIOUS) return PREBA_ERR_INVALID_ARG;
  if (batch->table_host) {
    rc = check_table(batch->table_host, batch->n, batch->pixels_bytes);
    if (rc != PREBA_OK) return rc;
    if (opt->crop_origin_host) {
      // every window must lie on its image's resized grid
      for (uint32_t i = 0; i < batch->n; ++i) {
        const uint64_t h = batch->table_host[i].h, w = batch->table_host[i].w;
        const uint64_t rl = opt->resize_short * (h > w ? h : w) / (h > w ? w : h);
        const uint64_t rh = h <= w ? opt->resize_short : rl, rw = h <= w ? rl : opt->resize_short;
        if (opt->crop_origin_host[2 * i] + static_cast<uint64_t>(opt->out_size) > rh ||
            opt->crop_origin_host[2 * i + 1] + static_cast<uint64_t>(opt->out_size) > rw)
          return PREBA_ERR_BAD_CROP;
      }
    }
  }
  Params p = make_params(batch->pixels, batch->pixels_bytes, batch->table, batch->n, batch->out,
                         batch->status, batch->scratch, opt->out_size, opt->resize_short,
                         opt->mean, opt->std);
  p.crop = opt->crop_origin;
  const int mode = opt->out_dtype == PREBA_U8 ? kU8 : (round_u8 ? kRoundFloat : kFloat);
  return launch(p, opt->out_dtype, (batch->flags & PREBA_OVERLAP_PREVIOUS) != 0,
                static_cast<cudaStream_t>(stream), mode);
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
                        dtype_bytes(out_dtype);
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
  rc = launch(p, out_dtype, false, s);
  if (rc != PREBA_OK) return rc;
  err = cudaMemcpyAsync(b->out_host, b->dev_out, need, cudaMemcpyDeviceToHost, s);
  if (err != cudaSuccess) {
    g_last_cuda_error = static_cast<int>(err);
    return PREBA_ERR_CUDA;
  }
  return PREBA_OK;
}

extern "C" int preba_preprocess_images(const preba_image_batch_t* b, uint32_t out_size,
                                       uint32_t resize_short, const float mean[3],
                                       const float std[3], int out_dtype, void* stream) {
  using namespace preba;
  if (!b || !b->images || !b->h || !b->w || !b->table_host || !b->out_host || !b->dev_table ||
      b->n == 0 || (b->flags & ~(PREBA_IMAGES_IN_PLACE | PREBA_IMAGES_OUT_IN_PLACE)))
    return PREBA_ERR_INVALID_ARG;
  const bool in_place = (b->flags & PREBA_IMAGES_IN_PLACE) != 0;
  // the kernel stores the result in (pinned) host memory itself instead of a copy afterwards
  const bool out_in_place = (b->flags & PREBA_IMAGES_OUT_IN_PLACE) != 0;
  void* const out = out_in_place ? b->out_host : b->dev_out;
  for (uint32_t i = 0; i < b->n; ++i)
    if (!b->images[i] || !dims_ok(b->h[i], b->w[i])) return PREBA_ERR_INVALID_ARG;
  const uint8_t* pixels = b->dev_pixels;
  uint64_t pixels_bytes = 0;
  if (in_place) {
    // the "packed buffer" is host memory as it stands: offsets from the lowest image
    uintptr_t lo = UINTPTR_MAX;
    for (uint32_t i = 0; i < b->n; ++i) {
      const uintptr_t a = reinterpret_cast<uintptr_t>(b->images[i]);
      if (a % PREBA_PACK_ALIGN) return PREBA_ERR_INVALID_ARG;
      lo = a < lo ? a : lo;
    }
    for (uint32_t i = 0; i < b->n; ++i) {
      const uint64_t off = reinterpret_cast<uintptr_t>(b->images[i]) - lo;
      b->table_host[i].offset = off;
      b->table_host[i].h = b->h[i];
      b->table_host[i].w = b->w[i];
      const uint64_t end = off + align_up(3ull * b->h[i] * b->w[i], 16);
      pixels_bytes = end > pixels_bytes ? end : pixels_bytes;
    }
    pixels = reinterpret_cast<const uint8_t*>(lo);
  } else {
    // the packed layout: running byte count rounded up to the alignment
    uint64_t at = 0;
    for (uint32_t i = 0; i < b->n; ++i) {
      b->table_host[i].offset = at;
      b->table_host[i].h = b->h[i];
      b->table_host[i].w = b->w[i];
      at = align_up(at + 3ull * b->h[i] * b->w[i], PREBA_PACK_ALIGN);
    }
    pixels_bytes = at;
    if (b->dev_pixels_bytes < pixels_bytes) return PREBA_ERR_BUFFER_TOO_SMALL;
  }
  int rc = check_args(pixels, pixels_bytes, b->dev_table, b->n, out, b->out_bytes,
                      out_size, resize_short, mean, std, out_dtype);
  if (rc != PREBA_OK) return rc;
  if (reinterpret_cast<uintptr_t>(b->dev_scratch) % 16) return PREBA_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const uint64_t need = static_cast<uint64_t>(b->n) * 3ull * out_size * out_size *
                        dtype_bytes(out_dtype);
  cudaError_t err = cudaSuccess;
  if (out_in_place) {
    // the device must be able to address the result buffer through the pointer given
    cudaPointerAttributes attr;
    err = cudaPointerGetAttributes(&attr, b->out_host);
    if (err == cudaSuccess && (attr.type == cudaMemoryTypeUnregistered ||
                               attr.devicePointer != b->out_host))
      return PREBA_ERR_INVALID_ARG;
  }
  if (in_place) {
    // the device must be able to address the images through the pointers given
    for (uint32_t i = 0; i < b->n && err == cudaSuccess; ++i) {
      cudaPointerAttributes attr;
      err = cudaPointerGetAttributes(&attr, b->images[i]);
      if (err == cudaSuccess && (attr.type == cudaMemoryTypeUnregistered ||
                                 attr.devicePointer != static_cast<const void*>(b->images[i])))
        return PREBA_ERR_INVALID_ARG;
    }
  } else {
    for (uint32_t i = 0; i < b->n && err == cudaSuccess; ++i)
      err = cudaMemcpyAsync(b->dev_pixels + b->table_host[i].offset, b->images[i],
                            3ull * b->h[i] * b->w[i], cudaMemcpyHostToDevice, s);
  }
  if (err == cudaSuccess)
    err = cudaMemcpyAsync(b->dev_table, b->table_host, sizeof(preba_img_t) * b->n,
                          cudaMemcpyHostToDevice, s);
  if (err != cudaSuccess) {
    g_last_cuda_error = static_cast<int>(err);
    return PREBA_ERR_CUDA;
  }
  const Params p = make_params(pixels, pixels_bytes, b->dev_table, b->n, out, b->dev_status,
                               b->dev_scratch, out_size, resize_short, mean, std);
  rc = launch(p, out_dtype, false, s);
  if (rc != PREBA_OK) return rc;
  if (!out_in_place) err = cudaMemcpyAsync(b->out_host, b->dev_out, need, cudaMemcpyDeviceToHost, s);
  if (err != cudaSuccess) {
    g_last_cuda_error = static_cast<int>(err);
    return PREBA_ERR_CUDA;
  }
  return PREBA_OK;
}

extern "C" int preba_preprocess_repeated(const preba_batch_t* batch, uint32_t out_size,
                                         uint32_t resize_short, const float mean[3],
                                         const float std[3], int out_dtype, void* stream,
                                         uint32_t iterations, float* latency_us,
                                         float* span_ms) {
  using namespace preba;
  if (!batch || iterations == 0) return PREBA_ERR_INVALID_ARG;
  int rc = check_args(batch->pixels, batch->pixels_bytes, batch->table, batch->n, batch->out,
                      batch->out_bytes, out_size, resize_short, mean, std, out_dtype);
  if (rc != PREBA_OK) return rc;
  if (reinterpret_cast<uintptr_t>(batch->scratch) % 16) return PREBA_ERR_INVALID_ARG;
  if (batch->flags & ~PREBA_OVERLAP_PREVIOUS) return PREBA_ERR_INVALID_ARG;
  if (batch->table_host) {
    rc = check_table(batch->table_host, batch->n, batch->pixels_bytes);
    if (rc != PREBA_OK) return rc;
  }
  const Params p = make_params(batch->pixels, batch->pixels_bytes, batch->table, batch->n,
                               batch->out, batch->status, batch->scratch, out_size, resize_short,
                               mean, std);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const bool overlap = (batch->flags & PREBA_OVERLAP_PREVIOUS) != 0;
  std::vector<cudaEvent_t> ev(2 * static_cast<size_t>(iterations), nullptr);
  cudaError_t err = cudaSuccess;
  for (auto& e : ev) {
    err = cudaEventCreate(&e);
    if (err != cudaSuccess) break;
  }
  rc = PREBA_OK;
  for (uint32_t i = 0; i < iterations && err == cudaSuccess && rc == PREBA_OK; ++i) {
    err = cudaEventRecord(ev[2 * i], s);
    if (err == cudaSuccess) rc = launch(p, out_dtype, overlap, s);
    if (err == cudaSuccess && rc == PREBA_OK) err = cudaEventRecord(ev[2 * i + 1], s);
  }
  if (err == cudaSuccess) err = cudaStreamSynchronize(s);
  if (err == cudaSuccess && rc == PREBA_OK) {
    for (uint32_t i = 0; i < iterations && latency_us && err == cudaSuccess; ++i) {
      float ms = 0.f;
      err = cudaEventElapsedTime(&ms, ev[2 * i], ev[2 * i + 1]);
      latency_us[i] = ms * 1000.0f;
    }
    if (span_ms && err == cudaSuccess)
      err = cudaEventElapsedTime(span_ms, ev[0], ev[2 * static_cast<size_t>(iterations) - 1]);
  }
  for (auto& e : ev)
    if (e) cudaEventDestroy(e);
  if (rc != PREBA_OK) return rc;
  if (err != cudaSuccess) {
    g_last_cuda_error = static_cast<int>(err);
    return PREBA_ERR_CUDA;
  }
  return PREBA_OK;
}

namespace preba {

// One warp waits on a barrier nobody arrives at: the wait runs out and reports.
__global__ void __launch_bounds__(32) preba_wait_limit_kernel(int32_t* status) {
  __shared__ uint64_t never;
  if (threadIdx.x == 0) {
    mbar_init(smem_addr(&never), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncwarp();
  if (!mbar_wait(smem_addr(&never), 0) && threadIdx.x == 0) report(status, PREBA_ERR_TIMEOUT);
}

}  // namespace preba

extern "C" int preba_selftest_wait_limit(int32_t* status, void* stream) {
  if (!status) return PREBA_ERR_INVALID_ARG;
  preba::preba_wait_limit_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(status);
  const cudaError_t err = cudaGetLastError();
  if (err != cudaSuccess) {
    preba::g_last_cuda_error = static_cast<int>(err);
    return PREBA_ERR_CUDA;
  }
  return PREBA_OK;
}

// ---- host-to-host without any allocation ------------------------------------------------------------
//
// Staging space that ships with the library: every GPU that loads it carries this array
// until the process exits.  In host code the symbol is only a stand-in; its device address
// comes from cudaGetSymbolAddress, once per device.
static __device__ __align__(256) unsigned char g_noalloc_space[PREBA_NOALLOC_MAX_BYTES];

namespace preba {

constexpr uint64_t kNoallocCounters = 0;   // scheduling counters (PREBA_SCRATCH_BYTES)
constexpr uint64_t kNoallocStatus = 256;   // status word
constexpr uint64_t kNoallocHeader = 512;   // cleared at the start of every call

// Device address of the staging array on the current device; looked up on the first call
// per device (concurrent first calls store the same value).
cudaError_t noalloc_base(unsigned char** base) {
  constexpr int kMaxDevices = 64;
  static std::atomic<unsigned char*> cache[kMaxDevices];
  int dev = 0;
  cudaError_t err = cudaGetDevice(&dev);
  if (err != cudaSuccess) return err;
  if (dev >= 0 && dev < kMaxDevices) {
    unsigned char* known = cache[dev].load(std::memory_order_acquire);
    if (known) {
      *base = known;
      return cudaSuccess;
    }
  }
  void* ptr = nullptr;
  err = cudaGetSymbolAddress(&ptr, g_noalloc_space);
  if (err != cudaSuccess) return err;
  *base = static_cast<unsigned char*>(ptr);
  if (dev >= 0 && dev < kMaxDevices) cache[dev].store(*base, std::memory_order_release);
  return cudaSuccess;
}

}  // namespace preba

extern "C" int preba_preprocess_host_noalloc(const uint8_t* packed_host, uint64_t packed_bytes,
                                             const preba_img_t* table_host, uint32_t n,
                                             void* out_host, uint64_t out_bytes,
                                             int32_t* status_host, uint32_t out_size,
                                             uint32_t resize_short, const float mean[3],
                                             const float std[3], int out_dtype, void* stream) {
  using namespace preba;
  if (!packed_host || !table_host || !out_host) return PREBA_ERR_INVALID_ARG;
  // argument checks of the device entry points, with stand-in addresses for the staging
  int rc = check_args(reinterpret_cast<const uint8_t*>(uintptr_t{256}), packed_bytes,
                      reinterpret_cast<const void*>(uintptr_t{256}), n,
                      reinterpret_cast<const void*>(uintptr_t{256}), out_bytes, out_size,
                      resize_short, mean, std, out_dtype);
  if (rc != PREBA_OK) return rc;
  rc = check_table(table_host, n, packed_bytes);
  if (rc != PREBA_OK) return rc;
  const uint64_t need_out = static_cast<uint64_t>(n) * 3ull * out_size * out_size *
                            dtype_bytes(out_dtype);
  const uint64_t table_bytes = static_cast<uint64_t>(n) * sizeof(preba_img_t);
  // each part alone first, so that the sums below cannot wrap
  if (packed_bytes > PREBA_NOALLOC_MAX_BYTES || need_out > PREBA_NOALLOC_MAX_BYTES ||
      table_bytes > PREBA_NOALLOC_MAX_BYTES)
    return PREBA_ERR_TOO_LARGE;
  const uint64_t at_table = kNoallocHeader;
  const uint64_t at_pixels = at_table + align_up(table_bytes, 256);
  const uint64_t at_out = at_pixels + align_up(packed_bytes, 256);
  const uint64_t total = at_out + align_up(need_out, 256);
  if (total > PREBA_NOALLOC_MAX_BYTES) return PREBA_ERR_TOO_LARGE;

  unsigned char* base = nullptr;
  cudaError_t err = noalloc_base(&base);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (err == cudaSuccess) err = cudaMemsetAsync(base, 0, kNoallocHeader, s);
  if (err == cudaSuccess)
    err = cudaMemcpyAsync(base + at_pixels, packed_host, packed_bytes, cudaMemcpyHostToDevice, s);
  if (err == cudaSuccess)
    err = cudaMemcpyAsync(base + at_table, table_host, table_bytes, cudaMemcpyHostToDevice, s);
  if (err != cudaSuccess) {
    g_last_cuda_error = static_cast<int>(err);
    return PREBA_ERR_CUDA;
  }
  const Params p = make_params(base + at_pixels, packed_bytes,
                               reinterpret_cast<const preba_img_t*>(base + at_table), n,
                               base + at_out, reinterpret_cast<int32_t*>(base + kNoallocStatus),
                               reinterpret_cast<uint32_t*>(base + kNoallocCounters), out_size,
                               resize_short, mean, std);
  rc = launch(p, out_dtype, false, s);
  if (rc != PREBA_OK) return rc;
  err = cudaMemcpyAsync(out_host, base + at_out, need_out, cudaMemcpyDeviceToHost, s);
  if (err == cudaSuccess && status_host)
    err = cudaMemcpyAsync(status_host, base + kNoallocStatus, sizeof(int32_t),
                          cudaMemcpyDeviceToHost, s);
  if (err != cudaSuccess) {
    g_last_cuda_error = static_cast<int>(err);
    return PREBA_ERR_CUDA;
  }
  return PREBA_OK;
}

extern "C" int preba_last_cuda_error(void) { return preba::g_last_cuda_error; }
