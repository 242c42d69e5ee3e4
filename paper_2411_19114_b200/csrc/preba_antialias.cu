// Antialiased Resize -> Crop -> Normalize (the Resize unit of the paper's Table 1 reconfigured,
// Sec. 4.2 "Flexible design based on reconfigurable hardware", for inputs much larger than the
// model's resolution): a separable triangle filter whose half-width is the reduction factor.
//
// On each axis, with n_in input pixels and R resized pixels, M = max(n_in, R):
//   weight of input pixel j for resized pixel X  =  W / sum W,
//   W = max(0, 2M - |(2j+1) R - (2X+1) n_in|)        (an integer; the triangle times 2M)
// so taps and un-normalised weights come from exact integer arithmetic; the sums run in fp32.
//
// Three kernels share a batch, chosen per image by mm2_plan and mma_plan below: one with both
// passes on the tensor cores (images reduced more than 2.5 times vertically), one with the
// horizontal pass on them, and the general one described next; each skips the others' images.
//
// The general kernel: one CTA produces `rows` consecutive output rows of one image, two at a
// time (neighbouring rows share about half of their input rows).  Per pair of output rows:
//   vertical pass   every thread owns up to kWords 4-byte words of the needed byte range of
//                   the input rows and accumulates them into both rows' sums, all loads of a
//                   row in flight together; the results go to shared memory, one plane per
//                   channel and row, one element of padding every 32 so that the strided reads
//                   below spread over the banks;
//   horizontal pass a thread per output column sums its taps for the three channels of both
//                   rows, applies the normalising multiply-add and stores the elements.
// The horizontal weights are the same for every row of the image, so they are tabulated once
// per CTA in shared memory.  HBM traffic is every input byte under the crop's footprint once
// (rows shared by neighbouring CTAs come from L2) plus the output.
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "preba.h"
#include "preba_internal.h"

namespace preba {
namespace aa {

constexpr int kThreads = 256;
constexpr uint32_t kMaxRows = 32;  // output rows per CTA, at most
constexpr uint32_t kWords = 3;     // 4-byte words of a row a thread holds at a time

struct Params {
  const uint8_t* pixels;
  uint64_t pixels_bytes;
  const preba_img_t* table;
  const uint32_t* crop;  // 2n (top, left) or nullptr
  void* out;
  int32_t* status;
  uint32_t n, C, S;
  uint32_t rows;         // output rows per CTA
  uint32_t smem_floats;  // shared memory the launch carries, in 4-byte units
  uint32_t mma_rows;     // output rows per CTA of the tensor-core kernel (<= kMmaRows)
  uint32_t mma_smem;     // bytes of shared memory of the tensor-core kernel's launch; images it
                         // can take (mma_plan) are left to it by the other kernel.  0: none are
  uint32_t mm2_rows;     // the same two for the kernel with both passes on the tensor cores
  uint32_t mm2_smem;     // (mm2_plan), which comes first in the choice
  float mul[3], add[3];  // y = v * mul + add
};

// One axis of one image.
struct Axis {
  uint32_t n_in, R, M;  // M = max(n_in, R)
  uint32_t taps;        // upper bound of the taps of one resized pixel
};

__host__ __device__ inline Axis make_axis(uint32_t n_in, uint32_t R) {
  Axis a;
  a.n_in = n_in;
  a.R = R;
  a.M = n_in > R ? n_in : R;
  // (2j+1) R lies strictly inside an interval of length 4M: fewer than 2M/R + 1 values of j
  a.taps = 2u * a.M / R + 2u;
  return a;
}

// Whether the un-normalised weights fit 16 bits and a row's weighted byte sum 32 bits, so that
// the vertical pass can run on integer dot products.
__host__ __device__ inline bool integer_weights_fit(const Axis& a) {
  return 2ull * a.M <= 65535ull && 255ull * a.taps * 2ull * a.M < (1ull << 32);
}

__host__ __device__ inline int64_t floor_div(int64_t a, int64_t b) {  // b > 0
  const int64_t q = a / b;
  return (a % b != 0 && a < 0) ? q - 1 : q;
}

// First tap and one past the last tap of resized pixel X (those with W > 0, inside the image).
__host__ __device__ inline void tap_range(const Axis& a, uint32_t X, uint32_t* lo, uint32_t* hi) {
  const int64_t centre = static_cast<int64_t>(2ull * X + 1) * a.n_in;
  const int64_t R = a.R, M2 = 2ll * a.M;
  // (2j+1) R > centre - 2M  <=>  j > (centre - 2M - R) / 2R
  int64_t first = floor_div(centre - M2 - R, 2 * R) + 1;
  // (2j+1) R < centre + 2M  <=>  j < (centre + 2M - R) / 2R
  int64_t last = floor_div(centre + M2 - R + 2 * R - 1, 2 * R);  // ceiling: one past the last
  if (first < 0) first = 0;
  if (last > static_cast<int64_t>(a.n_in)) last = a.n_in;
  *lo = static_cast<uint32_t>(first);
  *hi = static_cast<uint32_t>(last);
}

// Un-normalised integer weight of input pixel j for resized pixel X (positive inside tap_range).
__host__ __device__ inline int32_t tap_weight(const Axis& a, uint32_t X, uint32_t j) {
  const int64_t d = static_cast<int64_t>(2ull * j + 1) * a.R -
                    static_cast<int64_t>(2ull * X + 1) * a.n_in;
  const int64_t w = 2ll * a.M - (d < 0 ? -d : d);
  return w > 0 ? static_cast<int32_t>(w) : 0;
}

__host__ __device__ inline void resized_size(uint32_t h, uint32_t w, uint32_t S, uint32_t* rh,
                                             uint32_t* rw) {
  if (h <= w) {
    *rh = S;
    *rw = static_cast<uint32_t>(static_cast<uint64_t>(S) * w / h);
  } else {
    *rh = static_cast<uint32_t>(static_cast<uint64_t>(S) * h / w);
    *rw = S;
  }
}

// Shared-memory plan of one CTA (in 4-byte units), from bounds that hold for any crop origin.
// Output rows are made two at a time: neighbouring rows share about half of their input rows.
struct Plan {
  uint32_t tx;     // pitch of the horizontal weight table (odd: table reads spread over banks)
  uint32_t tp;     // pitch, in (weight of row a, weight of row b) pairs, of the row-pair tables
  uint32_t plane;  // elements of one channel plane of the vertical pass's result
  uint32_t ti;     // pitch of the integer row-pair tables: an entry per two input rows
  uint32_t off_wx, off_xlo, off_xcnt, off_wp, off_wi, off_inv, off_plo, off_pcnt, off_v, off_ring;
  uint32_t seg;    // bytes of one slot of the ring of staged input rows
};

__host__ __device__ inline Plan make_plan(const Axis& ax, const Axis& ay, uint32_t C,
                                          uint32_t rows) {
  Plan p;
  p.tx = ax.taps | 1u;
  // taps of one row plus the distance between the first taps of neighbouring rows
  p.tp = ay.taps + ay.M / ay.R + 2u;
  // pixels under C resized pixels: ((C-1) n_in + 2M)/R + 2 <= (C+1) M/R + 2; one pixel before
  // and two after for the word-aligned ends
  const uint64_t span = (static_cast<uint64_t>(C + 1) * ax.M + ax.R - 1) / ax.R + 2 + 4;
  const uint32_t px = static_cast<uint32_t>(span < ax.n_in + 4ull ? span : ax.n_in + 4ull);
  p.plane = px + px / 32 + 1;
  const uint32_t pairs = (rows + 1) / 2;
  uint32_t at = 0;
  p.off_wx = at, at += C * p.tx;
  p.off_xlo = at, at += C;
  p.off_xcnt = at, at += C;
  at += at & 1u;  // the pair table is read 8 bytes at a time
  p.off_wp = at, at += pairs * p.tp * 2;
  p.ti = (p.tp + 1u) / 2u;
  p.off_wi = at, at += pairs * p.ti * 2;
  p.off_inv = at, at += pairs * 2;
  p.off_plo = at, at += pairs;
  p.off_pcnt = at, at += pairs;
  p.off_v = at, at += 6 * p.plane;
  at = (at + 3u) & ~3u;  // the ring of staged input rows starts on a 16-byte boundary
  p.off_ring = at;
  // a staged row: the needed bytes from a 16-byte boundary of global memory, a multiple of 16
  p.seg = (3u * px + 32u + 15u) & ~15u;
  return p;
}

// Slots of the ring that `floats` 4-byte units of shared memory leave room for (each slot: a
// staged row and its 8-byte barrier).
__host__ __device__ inline uint32_t ring_slots(const Plan& p, uint32_t floats) {
  return floats <= p.off_ring ? 0u : (floats - p.off_ring) * 4u / (p.seg + 8u);
}

// Shared memory (4-byte units) for a ring of `slots` rows.
__host__ __device__ inline uint64_t plan_floats(const Plan& p, uint64_t slots) {
  return p.off_ring + (slots * (p.seg + 8ull) + 3ull) / 4ull;
}

// ---- which images the tensor-core kernel (further down) takes ------------------------------------

constexpr uint32_t kMmaRows = 256;    // output rows per CTA, at most
constexpr uint32_t kGroup = 64;       // output columns per CTA (32 tiles of two)
constexpr uint32_t kTileBytes = 64;   // bytes of an input row one tile multiplies (two k-steps)
constexpr uint32_t kMaxTapsX = 20;    // horizontal taps of one column, at most
constexpr uint32_t kMaxTapsY = 24;    // vertical taps of one row, at most
constexpr uint32_t kHPlane = 66;      // floats between the channel planes of a row of H
constexpr uint32_t kHPitch = 200;     // floats between rows of H (3 planes and padding: a warp's
                                      // stores and loads spread over the banks)
constexpr uint32_t kHFloats = 16u * kHPitch;  // one tile of H; the kernel keeps two
constexpr uint32_t kMmaThreads = 256;

struct MmaPlan {
  uint32_t seg;      // bytes of one staged input row in the ring
  uint32_t slots;    // 16-row slots of the ring
  uint32_t off_ring; // byte offsets into the dynamic shared memory
  uint32_t off_h, off_wx, off_xlo, off_xcnt, off_invx, off_wy, off_ylo, off_ycnt, off_bar;
};

// Whether the tensor-core kernel takes an image, and its shared-memory layout if so.  The same
// function decides in both kernels and on the host.
__host__ __device__ inline bool mma_plan(const Axis& ax, const Axis& ay, uint32_t w, uint32_t C,
                                         uint32_t smem_bytes, MmaPlan* out) {
  if (smem_bytes == 0 || (w & 3u) != 0) return false;  // rows must start on the same byte phase
  if (ax.M > 32767u) return false;                      // weights in two bytes
  const uint32_t step = (ax.n_in + ax.R - 1u) / ax.R;   // first taps of neighbours differ by <= step
  if (ax.taps > kMaxTapsX || 3u * (ax.taps + step) + 3u > kTileBytes) return false;
  if (255ull * ax.taps * 2ull * ax.M >= (1ull << 31)) return false;  // 32-bit sums
  if (ay.taps > kMaxTapsY || ay.M > 32767u) return false;
  // a warp finishes an output row before the row 32 further down begins: not for enlargements
  // beyond about six times
  if (32ull * ay.n_in < 5ull * ay.R) return false;
  const uint32_t cols = C < kGroup ? C : kGroup;
  // pixels under a group: first taps at most ceil((cols - 1) n_in / R) + 1 apart, plus one
  // column's taps
  const uint64_t px = (static_cast<uint64_t>(cols - 1u) * ax.n_in + ax.R - 1u) / ax.R + ax.taps + 3u;
  MmaPlan p;
  // a staged row: up to 15 bytes of skew, the bytes under the group, the overshoot of the last
  // tile; 16 modulo 128, so that the eight rows a warp reads together lie four banks apart
  p.seg = static_cast<uint32_t>(((16u + 3u * px + kTileBytes + 111u) & ~127ull) + 16u);
  uint32_t at = 0;
  p.off_h = at, at += 2u * kHFloats * 4u;
  p.off_wx = at, at += kGroup * kMaxTapsX * 2u;
  p.off_xlo = at, at += kGroup * 4u;
  p.off_xcnt = at, at += kGroup * 4u;
  p.off_invx = at, at += kGroup * 4u;
  p.off_wy = at, at += kMmaRows * kMaxTapsY * 4u;
  p.off_ylo = at, at += kMmaRows * 4u;
  p.off_ycnt = at, at += kMmaRows * 4u;
  p.off_bar = at, at += 64u;
  at = (at + 15u) & ~15u;
  p.off_ring = at;
  if (smem_bytes <= at) return false;
  const uint64_t room = (smem_bytes - at) / (16ull * p.seg);
  if (room < 2) return false;
  p.slots = room > 4 ? 4u : static_cast<uint32_t>(room);
  if (out) *out = p;
  return true;
}

// ---- both passes on the tensor cores ----------------------------------------------------------------
//
// For images reduced more than 2.5 times vertically the vertical pass is a matrix product too,
// and chaining it to the horizontal one keeps H out of shared memory altogether.  The
// horizontal product is taken transposed: the integer weights of five resized pixels x three
// channels are the A operand (16 rows, one unused; built once per warp, in registers), the
// bytes of eight input rows the B operand, again exactly as the rows lie in the ring, so a lane
// ends up with H[(x, ch)][input row] for (x, ch) = g, g + 8 and rows 2q, 2q + 1 of each
// eight: the layout an A operand has, with the input rows as its k index.  H is an exact
// integer below 2^24; its three bytes become three binary16 A operands (exact, scaled by
// powers of two), the integer weights of the (at most eight) output rows that lie under the
// sixteen input rows, split into two bytes, the binary16 B operands, and six more matrix
// instructions add the byte products into one fp32 accumulator.  An output row whose last
// tap has passed is normalised and stored.
// Fifteen warps each own one tile of five pixels from the ring to the store; the sixteenth
// feeds them: it issues the copies of a tile's rows and works out what is the same for every
// warp (the weights of the second product, which rows the tile completes) into the slot's
// record.  There is no CTA-wide barrier after the start, only the ring's full and empty
// barriers.
constexpr uint32_t kT2Px = 5;                        // resized pixels of an M-tile
constexpr uint32_t kT2Tiles = 15;                    // M-tiles of a CTA, one per consumer warp
constexpr uint32_t kT2Group = kT2Px * kT2Tiles;      // output columns per CTA
constexpr uint32_t kT2MaxSlots = 8;                  // 16-row slots of the ring, at most
constexpr uint32_t kT2Threads = 32 * (kT2Tiles + 1); // the last warp feeds the others
constexpr uint32_t kT2MetaBytes = 1024;              // per slot: what the feeding warp works out
                                                     // for a tile (32 bytes per lane)

struct Mm2Plan {
  uint32_t seg;    // bytes of one staged input row in the ring
  uint32_t slots;  // 16-row slots of the ring
  uint32_t ks;     // 32-byte steps of an M-tile's window (3 or 4)
  uint32_t off_wx, off_xlo, off_xcnt, off_invx, off_ylo, off_yhi, off_invy, off_bar, off_meta,
      off_ring;
};

// Whether the kernel with both passes on the tensor cores takes an image, and its
// shared-memory layout if so.  The same function decides in every kernel and on the host.
__host__ __device__ inline bool mm2_plan(const Axis& ax, const Axis& ay, uint32_t w, uint32_t C,
                                         uint32_t smem_bytes, Mm2Plan* out) {
  if (smem_bytes == 0 || (w & 3u) != 0) return false;  // rows must start on the same byte phase
  if (ax.M > 32767u || ay.M > 32767u) return false;    // weights in two bytes, 32-bit tap arithmetic
  if (ax.taps > kMaxTapsX || ay.taps > 32u) return false;
  if (255ull * ax.taps * 2ull * ax.M >= (1ull << 24)) return false;  // H in three bytes
  // at most eight output rows have taps among sixteen input rows: floor(15 R / n_in) + 3 <= 8
  if (ay.n_in <= ay.R || 15ull * ay.R / ay.n_in + 3ull > 8ull) return false;
  // the bytes of a row under an M-tile: first taps of its pixels at most ceil(4 n_in / R) + 1
  // apart, one pixel's taps, three bytes of alignment
  const uint64_t px_tile = (4ull * ax.n_in + ax.R - 1u) / ax.R + 1u + ax.taps;
  uint32_t ks = static_cast<uint32_t>((3ull * px_tile + 3u + 31u) / 32u);
  if (ks > 4u) return false;
  if (ks < 3u) ks = 3u;
  const uint32_t cols = C < kT2Group ? C : kT2Group;
  const uint64_t px = (static_cast<uint64_t>(cols - 1u) * ax.n_in + ax.R - 1u) / ax.R + ax.taps + 3u;
  Mm2Plan p;
  p.ks = ks;
  // a staged row: up to 15 bytes of skew, the bytes under the group, the overshoot of the last
  // window; 16 modulo 128, so that the eight rows a warp reads together lie four banks apart
  p.seg = static_cast<uint32_t>(((16u + 3u * px + 32u * ks + 111u) & ~127ull) + 16u);
  uint32_t at = 0;
  p.off_wx = at, at += kT2Group * kMaxTapsX * 2u;
  at = (at + 3u) & ~3u;
  p.off_xlo = at, at += kT2Group * 4u;
  p.off_xcnt = at, at += kT2Group * 4u;
  p.off_invx = at, at += kT2Group * 4u;
  p.off_ylo = at, at += kMmaRows * 4u;
  p.off_yhi = at, at += kMmaRows * 4u;
  p.off_invy = at, at += kMmaRows * 4u;
  at = (at + 7u) & ~7u;
  p.off_bar = at, at += 2u * kT2MaxSlots * 8u;
  at = (at + 15u) & ~15u;
  p.off_meta = at, at += kT2MaxSlots * kT2MetaBytes;
  p.off_ring = at;
  if (smem_bytes <= at) return false;
  const uint64_t room = (smem_bytes - at) / (16ull * p.seg);
  if (room < 2) return false;
  p.slots = room > kT2MaxSlots ? kT2MaxSlots : static_cast<uint32_t>(room);
  if (out) *out = p;
  return true;
}


__device__ __forceinline__ void report(int32_t* status, int code) {
  if (status) atomicCAS(status, 0, code);
}

template <typename OutT>
__device__ __forceinline__ OutT to_out(float v);
template <>
__device__ __forceinline__ float to_out<float>(float v) { return v; }
template <>
__device__ __forceinline__ __half to_out<__half>(float v) { return __float2half_rn(v); }
template <>
__device__ __forceinline__ __nv_bfloat16 to_out<__nv_bfloat16>(float v) {
  return __float2bfloat16_rn(v);
}

// Sum of the integer weights of taps j0 .. j1 - 1 of resized pixel X: the distance term moves
// by 2R from one tap to the next, so one 64-bit product starts the run.
__device__ __forceinline__ uint64_t weight_sum(const Axis& a, uint32_t X, uint32_t j0, uint32_t j1) {
  int64_t d = static_cast<int64_t>(2ull * j0 + 1) * a.R - static_cast<int64_t>(2ull * X + 1) * a.n_in;
  const int64_t two_m = 2ll * a.M, step = 2ll * a.R;
  uint64_t sum = 0;
  for (uint32_t j = j0; j < j1; ++j, d += step) sum += static_cast<uint64_t>(two_m - (d < 0 ? -d : d));
  return sum;
}

// Horizontal table: row q of `w` (pitch `pitch`) holds the normalised weights of resized
// pixel first + q from tap lo[q] on.
__device__ void tabulate(const Axis& a, uint32_t first, uint32_t count, uint32_t pitch, float* w,
                         uint32_t* lo, uint32_t* cnt) {
  for (uint32_t q = threadIdx.x; q < count; q += kThreads) {
    uint32_t j0, j1;
    tap_range(a, first + q, &j0, &j1);
    const float inv = 1.0f / static_cast<float>(weight_sum(a, first + q, j0, j1));
    int64_t d = static_cast<int64_t>(2ull * j0 + 1) * a.R -
                static_cast<int64_t>(2ull * (first + q) + 1) * a.n_in;
    const int64_t two_m = 2ll * a.M, step = 2ll * a.R;
    for (uint32_t j = j0; j < j1; ++j, d += step)
      w[q * pitch + (j - j0)] = static_cast<float>(two_m - (d < 0 ? -d : d)) * inv;
    lo[q] = j0;
    cnt[q] = j1 - j0;
  }
}

// Vertical tables: pair r covers resized rows first + 2r (a) and first + 2r + 1 (b, if below
// `count`); entry i of its table holds both rows' normalised weights of input row lo[r] + i
// (zero where a row does not reach), over the union of the two rows' taps.
// With `wi`: entry i / 2 of the pair's integer table packs the un-normalised 16-bit weights of
// input rows lo[r] + i (low half) and lo[r] + i + 1 (high half), .x for row a and .y for row b.
// inv[r] holds the reciprocals of the two rows' weight sums.  A thread per pair finds the
// ranges and the sums; after a barrier a thread per table entry writes the weights.
__device__ void tabulate_pairs(const Axis& a, uint32_t first, uint32_t count, uint32_t pitch,
                               float2* w, uint32_t* lo, uint32_t* cnt, uint32_t ipitch, uint2* wi,
                               float2* inv) {
  const uint32_t pairs = (count + 1) / 2;
  for (uint32_t r = threadIdx.x; r < pairs; r += kThreads) {
    const uint32_t ya = first + 2 * r;
    const bool has_b = 2 * r + 1 < count;
    uint32_t a0, a1, b0, b1;
    tap_range(a, ya, &a0, &a1);
    b0 = a0, b1 = a1;
    if (has_b) tap_range(a, ya + 1, &b0, &b1);
    lo[r] = a0;  // first taps do not decrease with the row
    cnt[r] = (a1 > b1 ? a1 : b1) - a0;
    inv[r] = make_float2(1.0f / static_cast<float>(weight_sum(a, ya, a0, a1)),
                         has_b ? 1.0f / static_cast<float>(weight_sum(a, ya + 1, b0, b1)) : 0.f);
  }
  __syncthreads();
  for (uint32_t at = threadIdx.x; at < pairs * pitch; at += kThreads) {
    const uint32_t r = at / pitch, i = at - r * pitch;
    if (i >= cnt[r]) continue;
    const uint32_t ya = first + 2 * r, j = lo[r] + i;
    const bool has_b = 2 * r + 1 < count;
    const float2 scale = inv[r];
    w[at] = make_float2(static_cast<float>(tap_weight(a, ya, j)) * scale.x,
                        has_b ? static_cast<float>(tap_weight(a, ya + 1, j)) * scale.y : 0.f);
  }
  if (!wi) return;
  for (uint32_t at = threadIdx.x; at < pairs * ipitch; at += kThreads) {
    const uint32_t r = at / ipitch, i = 2 * (at - r * ipitch);
    if (i >= cnt[r]) continue;
    const uint32_t ya = first + 2 * r, j = lo[r] + i;
    const bool has_b = 2 * r + 1 < count, two = i + 1 < cnt[r];
    const uint32_t a_lo = static_cast<uint32_t>(tap_weight(a, ya, j));
    const uint32_t a_hi = two ? static_cast<uint32_t>(tap_weight(a, ya, j + 1)) : 0u;
    const uint32_t b_lo = has_b ? static_cast<uint32_t>(tap_weight(a, ya + 1, j)) : 0u;
    const uint32_t b_hi = has_b && two ? static_cast<uint32_t>(tap_weight(a, ya + 1, j + 1)) : 0u;
    wi[at] = make_uint2(a_lo | (a_hi << 16), b_lo | (b_hi << 16));
  }
}

// ---- shared-memory barriers and bulk copies (PTX) -------------------------------------------

constexpr uint32_t kSpinLimit = 1u << 20;  // bounded waits: give up, report, leave

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

// The same, every try with a time hint: a thread whose phase is not complete yet is put aside
// by the hardware for up to about that long (or until the phase completes) instead of coming
// back at once, so waiting warps leave the issue slots to the others.
__device__ __forceinline__ bool mbar_wait_parked(uint32_t bar, uint32_t parity) {
  for (uint32_t it = 0; it < kSpinLimit; ++it) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity), "r"(4000u)
        : "memory");
    if (ok) return true;
  }
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

// Orders earlier shared-memory reads before later asynchronous-copy writes.
__device__ __forceinline__ void fence_async_shared() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// The ring of staged input rows of one CTA.  Row y of the image lives in slot (y - first) % slots
// from the time thread 0 issues its copy until every row below the next pair's first row is
// dead; the slot's barrier completes once per use, so use u of a slot is awaited with parity u & 1.
struct Ring {
  uint32_t data, bars;  // shared-memory addresses
  uint32_t slots, seg;
  uint32_t first;       // image row in use 0 of slot 0
  uint32_t issued;      // rows below this have been asked for (meaningful in thread 0)
  uint32_t end;         // one past the last row the CTA needs
  const uint8_t* image; // first byte of the image
  const uint8_t* stop;  // end of the last whole 16-byte unit of the pixel buffer
  uint64_t pitch;       // bytes per image row
  uint32_t b0, bytes;   // first needed byte of a row and the count of needed bytes
  int32_t* status;      // the launch's status word (for the checked build's reports)
};

// Thread 0: asks for every row below `limit` that has not been asked for.
__device__ __forceinline__ void ring_issue(Ring& rg, uint32_t limit) {
  if (limit > rg.end) limit = rg.end;
  for (; rg.issued < limit; ++rg.issued) {
    const uint32_t slot = (rg.issued - rg.first) % rg.slots;
    const uint8_t* src = rg.image + rg.issued * rg.pitch + rg.b0;
    const uint32_t skew = static_cast<uint32_t>(reinterpret_cast<uintptr_t>(src)) & 15u;
    uint32_t bytes = (skew + rg.bytes + 15u) & ~15u;
    if (bytes > static_cast<uint64_t>(rg.stop - (src - skew)))  // only padding is lost
      bytes = static_cast<uint32_t>(rg.stop - (src - skew));
    const uint32_t bar = rg.bars + 8u * slot;
    // checked build: the row lies in its slot and in the pixel buffer (a row that does not is
    // announced with no bytes, so that its wait still ends)
    if (!PREBA_IN_RANGE(rg.status, bytes <= rg.seg && slot < rg.slots && src - skew + bytes <= rg.stop))
      bytes = 0;
    mbar_arrive_expect_tx(bar, bytes);
    if (bytes) bulk_copy_g2s(rg.data + slot * rg.seg, src - skew, bytes, bar);
  }
}

// Adds one input row's four bytes per word, weighted for both output rows of the pair.
__device__ __forceinline__ void accumulate(float (&acc)[kWords][8], const uint32_t (&px)[kWords],
                                           const float2 w) {
#pragma unroll
  for (uint32_t k = 0; k < kWords; ++k) {
    const float f0 = static_cast<float>(px[k] & 0xffu);
    const float f1 = static_cast<float>((px[k] >> 8) & 0xffu);
    const float f2 = static_cast<float>((px[k] >> 16) & 0xffu);
    const float f3 = static_cast<float>(px[k] >> 24);
    acc[k][0] = fmaf(w.x, f0, acc[k][0]);
    acc[k][1] = fmaf(w.x, f1, acc[k][1]);
    acc[k][2] = fmaf(w.x, f2, acc[k][2]);
    acc[k][3] = fmaf(w.x, f3, acc[k][3]);
    acc[k][4] = fmaf(w.y, f0, acc[k][4]);
    acc[k][5] = fmaf(w.y, f1, acc[k][5]);
    acc[k][6] = fmaf(w.y, f2, acc[k][6]);
    acc[k][7] = fmaf(w.y, f3, acc[k][7]);
  }
}

template <typename OutT>
__global__ void __launch_bounds__(kThreads) preba_antialias_kernel(const Params p) {
  extern __shared__ __align__(16) float smem[];
  const uint32_t tid = threadIdx.x, C = p.C;
  const uint32_t groups = (C + p.rows - 1) / p.rows;
  const uint32_t img = blockIdx.x / groups;
  const uint32_t k0 = (blockIdx.x % groups) * p.rows;
  const preba_img_t e = p.table[img];
  // The entry is checked again here: a bad one is skipped and reported (uniform over the CTA).
  // Rows are fetched in 16-byte units, so the buffer counts up to its last whole unit.
  const uint64_t usable = p.pixels_bytes & ~15ull;
  if (e.h < 1 || e.w < 1 || e.h > PREBA_MAX_DIM || e.w > PREBA_MAX_DIM ||
      e.offset % PREBA_PACK_ALIGN != 0 || e.offset > usable ||
      3ull * e.h * e.w > usable - e.offset) {
    if (tid == 0) report(p.status, PREBA_ERR_BAD_TABLE);
    return;
  }
  uint32_t rh, rw, top, left;
  resized_size(e.h, e.w, p.S, &rh, &rw);
  if (p.crop) {
    top = p.crop[2 * img];
    left = p.crop[2 * img + 1];
    if (static_cast<uint64_t>(top) + C > rh || static_cast<uint64_t>(left) + C > rw) {
      if (tid == 0) report(p.status, PREBA_ERR_BAD_CROP);
      return;
    }
  } else {
    top = (rh - C) / 2;
    left = (rw - C) / 2;
  }
  const Axis ax = make_axis(e.w, rw), ay = make_axis(e.h, rh);
  if (mm2_plan(ax, ay, e.w, C, p.mm2_smem, nullptr) ||
      mma_plan(ax, ay, e.w, C, p.mma_smem, nullptr))
    return;  // a tensor-core kernel's image
  const Plan pl = make_plan(ax, ay, C, p.rows);
  if (pl.off_ring > p.smem_floats) {
    if (tid == 0) report(p.status, PREBA_ERR_TOO_LARGE);
    return;
  }
  // Input rows are staged in shared memory by bulk copies, and summed by integer dot products,
  // when a ring that holds the rows of one pair of output rows fits and the integer weights are
  // narrow enough; other images are read from global memory directly and summed in fp32.
  const uint32_t slots = ring_slots(pl, p.smem_floats);
  const bool staged = slots >= pl.tp && integer_weights_fit(ay);
  const uint32_t rows_here = C - k0 < p.rows ? C - k0 : p.rows;
  const uint32_t pairs_here = (rows_here + 1) / 2;
  float* wx = smem + pl.off_wx;
  uint32_t* xlo = reinterpret_cast<uint32_t*>(smem + pl.off_xlo);
  uint32_t* xcnt = reinterpret_cast<uint32_t*>(smem + pl.off_xcnt);
  float2* wp = reinterpret_cast<float2*>(smem + pl.off_wp);
  uint32_t* plo = reinterpret_cast<uint32_t*>(smem + pl.off_plo);
  uint32_t* pcnt = reinterpret_cast<uint32_t*>(smem + pl.off_pcnt);
  float* va = smem + pl.off_v;  // three planes of row a, then three of row b
  float* vb = va + 3 * pl.plane;
  const uint8_t* ring = reinterpret_cast<const uint8_t*>(smem + pl.off_ring);
  Ring rg;
  rg.data = smem_addr(ring);
  rg.bars = rg.data + slots * pl.seg;
  rg.slots = slots;
  rg.seg = pl.seg;
  rg.status = p.status;
  tabulate(ax, left, C, pl.tx, wx, xlo, xcnt);
  uint2* wi = reinterpret_cast<uint2*>(smem + pl.off_wi);
  float2* inv = reinterpret_cast<float2*>(smem + pl.off_inv);
  tabulate_pairs(ay, top + k0, rows_here, pl.tp, wp, plo, pcnt, pl.ti, staged ? wi : nullptr, inv);
  if (tid == 0 && staged) {
    for (uint32_t s = 0; s < slots; ++s) mbar_init(rg.bars + 8u * s, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  // the byte range of a row that the window's taps cover, from a 4-byte boundary of the row
  const uint32_t b0 = (3u * xlo[0]) & ~3u;
  const uint32_t b1 = 3u * (xlo[C - 1] + xcnt[C - 1]);
  const uint32_t nwords = (b1 - b0 + 3u) / 4u;
  const uint32_t p0 = b0 / 3u;  // the pixel that element 0 of a plane stands for
  {
    const uint32_t last = (b0 + 4u * nwords - 1u) / 3u - p0;
    // cannot happen within the plan's bounds
    if (last + (last >> 5) >= pl.plane ||
        (staged && ((15u + 4u * nwords + 15u) & ~15u) > pl.seg)) {
      if (tid == 0) report(p.status, PREBA_ERR_TOO_LARGE);
      return;
    }
  }
  rg.image = p.pixels + e.offset;
  rg.stop = p.pixels + usable;
  rg.pitch = 3ull * e.w;
  rg.b0 = b0;
  rg.bytes = 4u * nwords;
  rg.first = plo[0];
  rg.issued = rg.first;
  rg.end = plo[pairs_here - 1] + pcnt[pairs_here - 1];
  if (tid == 0 && staged) ring_issue(rg, rg.first + slots);
  OutT* out = static_cast<OutT*>(p.out) + static_cast<uint64_t>(img) * 3u * C * C;
  bool failed = false;

  for (uint32_t r = 0; r < pairs_here; ++r) {
    // ---- vertical pass: both rows of the pair from one sweep over the staged input rows ----
    const uint32_t y0 = plo[r], ny = pcnt[r];
    const float2* wq = wp + r * pl.tp;
    const uint32_t slot0 = staged ? (y0 - rg.first) % slots : 0u;
    const uint32_t use0 = staged ? (y0 - rg.first) / slots : 0u;
    for (uint32_t w0 = tid; w0 < nwords; w0 += kThreads * kWords) {
      float acc[kWords][8];
#pragma unroll
      for (uint32_t k = 0; k < kWords; ++k)
#pragma unroll
        for (uint32_t t = 0; t < 8; ++t) acc[k][t] = 0.f;
      if (staged) {
        // two input rows per step: their bytes are interleaved so that one two-way dot product
        // adds both rows' contributions to a byte position (16-bit weights, 32-bit sums, exact)
        uint32_t sum[kWords][8];
#pragma unroll
        for (uint32_t k = 0; k < kWords; ++k)
#pragma unroll
          for (uint32_t t = 0; t < 8; ++t) sum[k][t] = 0u;
        const uint2* wq2 = wi + r * pl.ti;
        uint32_t slot = slot0, use = use0;
        uint32_t skew = static_cast<uint32_t>(
            reinterpret_cast<uintptr_t>(rg.image + y0 * rg.pitch + b0));  // low bits are used
        const uint32_t step = static_cast<uint32_t>(rg.pitch);
        for (uint32_t i = 0; i < ny; i += 2) {
          // the second row of the last step of an odd count has weight zero: its slot is read
          // (whatever it holds) but not waited for
          uint32_t slot1 = slot + 1, use1 = use;
          if (slot1 == slots) slot1 = 0, ++use1;
          if (!failed) failed = !mbar_wait(rg.bars + 8u * slot, use & 1u);
          if (!failed && i + 1 < ny) failed = !mbar_wait(rg.bars + 8u * slot1, use1 & 1u);
          const uint2 w = wq2[i / 2];
          const uint32_t skew1 = skew + step;
          const uint32_t m0 = skew & 3u, m1 = skew1 & 3u;  // the same for every thread
          const uint32_t* src0 =
              reinterpret_cast<const uint32_t*>(ring + slot * pl.seg + (skew & 12u)) + w0;
          const uint32_t* src1 =
              reinterpret_cast<const uint32_t*>(ring + slot1 * pl.seg + (skew1 & 12u)) + w0;
#pragma unroll
          for (uint32_t k = 0; k < kWords; ++k) {
            if (!failed && w0 + k * kThreads < nwords) {
              uint32_t q0 = src0[k * kThreads], q1 = src1[k * kThreads];
              if (m0) q0 = __funnelshift_r(q0, src0[k * kThreads + 1], 8u * m0);
              if (m1) q1 = __funnelshift_r(q1, src1[k * kThreads + 1], 8u * m1);
              const uint32_t lo = __byte_perm(q0, q1, 0x5140);  // bytes 0 and 1 of both rows
              const uint32_t hi = __byte_perm(q0, q1, 0x7362);  // bytes 2 and 3 of both rows
              sum[k][0] = __dp2a_lo(w.x, lo, sum[k][0]);
              sum[k][1] = __dp2a_hi(w.x, lo, sum[k][1]);
              sum[k][2] = __dp2a_lo(w.x, hi, sum[k][2]);
              sum[k][3] = __dp2a_hi(w.x, hi, sum[k][3]);
              sum[k][4] = __dp2a_lo(w.y, lo, sum[k][4]);
              sum[k][5] = __dp2a_hi(w.y, lo, sum[k][5]);
              sum[k][6] = __dp2a_lo(w.y, hi, sum[k][6]);
              sum[k][7] = __dp2a_hi(w.y, hi, sum[k][7]);
            }
          }
          slot = slot1 + 1, use = use1;
          if (slot == slots) slot = 0, ++use;
          skew = skew1 + step;
        }
        const float2 scale = inv[r];
#pragma unroll
        for (uint32_t k = 0; k < kWords; ++k)
#pragma unroll
          for (uint32_t t = 0; t < 4; ++t) {
            acc[k][t] = static_cast<float>(sum[k][t]) * scale.x;
            acc[k][4 + t] = static_cast<float>(sum[k][4 + t]) * scale.y;
          }
      } else {
        const uint32_t* words = reinterpret_cast<const uint32_t*>(p.pixels);
        uint64_t at0 = e.offset + y0 * rg.pitch + b0 + 4ull * w0;  // first byte of the first word
#pragma unroll 2
        for (uint32_t i = 0; i < ny; ++i, at0 += rg.pitch) {
          const float2 w = wq[i];
          const uint32_t m = static_cast<uint32_t>(at0) & 3u;  // the same for every thread
          uint32_t px[kWords];
#pragma unroll
          for (uint32_t k = 0; k < kWords; ++k) {
            px[k] = 0u;
            if (w0 + k * kThreads < nwords) {
              const uint64_t aligned = at0 + 4ull * k * kThreads - m;
              if (aligned + 4 <= p.pixels_bytes) px[k] = __ldg(words + aligned / 4);
              if (m) {
                const uint32_t hi =
                    aligned + 8 <= p.pixels_bytes ? __ldg(words + aligned / 4 + 1) : 0u;
                px[k] = __funnelshift_r(px[k], hi, 8u * m);
              }
            }
          }
          accumulate(acc, px, w);
        }
      }
#pragma unroll
      for (uint32_t k = 0; k < kWords; ++k) {
        if (w0 + k * kThreads < nwords) {
#pragma unroll
          for (uint32_t t = 0; t < 4; ++t) {
            const uint32_t byte = b0 + 4u * (w0 + k * kThreads) + t;
            const uint32_t pix = byte / 3u, ch = byte - 3u * pix, rel = pix - p0;
            const uint32_t at = ch * pl.plane + rel + (rel >> 5);
            // checked build: the element lies in its channel plane
            if (PREBA_IN_RANGE(p.status, rel + (rel >> 5) < pl.plane && ch < 3u)) {
              va[at] = acc[k][t];
              vb[at] = acc[k][4 + t];
            }
          }
        }
      }
    }
    failed = __syncthreads_or(failed) != 0;  // from here on the same in every thread
    if (failed) break;
    // every row below the next pair's first row is dead: its slot takes a new row, which
    // arrives while the horizontal pass runs
    if (tid == 0 && staged && r + 1 < pairs_here) {
      fence_async_shared();
      ring_issue(rg, plo[r + 1] + slots);
    }
    // ---- horizontal pass, normalisation, store ----
    const bool has_b = 2 * r + 1 < rows_here;
    for (uint32_t X = tid; X < C; X += kThreads) {
      const uint32_t rel0 = xlo[X] - p0, nx = xcnt[X];
      const float* w = wx + X * pl.tx;
      float s[6] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
      // checked build: the column's taps lie in the planes and in its row of the weight table
      if (!PREBA_IN_RANGE(p.status, nx <= pl.tx && rel0 + nx + ((rel0 + nx) >> 5) <= pl.plane &&
                                        k0 + 2 * r < C))
        continue;
      for (uint32_t t = 0; t < nx; ++t) {
        uint32_t idx = rel0 + t;
        idx += idx >> 5;
        const float wt = w[t];
#pragma unroll
        for (uint32_t c = 0; c < 3; ++c) {
          s[c] = fmaf(wt, va[c * pl.plane + idx], s[c]);
          s[3 + c] = fmaf(wt, vb[c * pl.plane + idx], s[3 + c]);
        }
      }
      const uint64_t o = static_cast<uint64_t>(k0 + 2 * r) * C + X;
#pragma unroll
      for (uint32_t c = 0; c < 3; ++c) {
        const uint64_t oc = o + static_cast<uint64_t>(c) * C * C;
        out[oc] = to_out<OutT>(fmaf(s[c], p.mul[c], p.add[c]));
        if (has_b) out[oc + C] = to_out<OutT>(fmaf(s[3 + c], p.mul[c], p.add[c]));
      }
    }
    __syncthreads();
  }

  if (failed && tid == 0) {
    report(p.status, PREBA_ERR_TIMEOUT);
    // copies already asked for may still be landing in the ring: wait for them (bounded)
    // before the CTA retires
    const uint32_t from = rg.issued - rg.first > slots ? rg.issued - slots : rg.first;
    for (uint32_t y = from; y < rg.issued; ++y)
      (void)mbar_wait(rg.bars + 8u * ((y - rg.first) % slots), ((y - rg.first) / slots) & 1u);
  }
}


// ---- the tensor-core path ---------------------------------------------------------------------------
//
// The horizontal pass is a banded matrix product: H[row][(X, ch)] = sum_b p[row][b] W[b][(X, ch)],
// b the byte position in the input row (b = 3 j + ch), W the integer triangle weight of pixel j
// for resized pixel X.  It runs as integer matrix instructions (m16n8k32, 8-bit operands, 32-bit
// sums, exact): 16 input rows by 64 bytes of a row against the weights of two resized pixels
// times three channels (six of the eight columns), the weights split into their high and low
// bytes (two instructions per 32 bytes, joined by a shift of the high sums).  The input rows
// are the A operand exactly as they lie in memory, so no byte is shuffled; the weights are the
// B operand, built once per warp and kept in registers.  The vertical pass then runs in fp32 on
// the 16 x 192 tile of H a CTA has just made (shared memory): output row y of the CTA belongs
// to warp y % 8, a lane has two columns per channel, and a warp adds the tile's rows under the
// taps of the rows it has in progress; a row whose last tap has passed is normalised and
// stored.
//
// A CTA makes up to kMmaRows output rows by kGroup columns of one image in one sweep over the
// input rows underneath, sixteen at a time, through a ring of bulk copies.

__device__ __forceinline__ void mma_u8(int32_t (&d)[4], const uint32_t (&a)[4], uint32_t b0,
                                       uint32_t b1) {
  asm("mma.sync.aligned.m16n8k32.row.col.s32.u8.u8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
      "{%0,%1,%2,%3};"
      : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// Taps of resized pixel X on an axis the tensor-core kernel admits (M <= 32767, so every term
// fits 32 bits): [lo, hi), as tap_range.
__device__ __forceinline__ void tap_range32(const Axis& a, uint32_t X, uint32_t* lo, uint32_t* hi) {
  const uint32_t centre = (2u * X + 1u) * a.n_in, m2 = 2u * a.M, r2 = 2u * a.R;
  const uint32_t first = centre >= m2 + a.R ? (centre - m2 - a.R) / r2 + 1u : 0u;
  const uint32_t last = (centre + m2 + a.R - 1u) / r2;
  *lo = first;
  *hi = last < a.n_in ? last : a.n_in;
}

__device__ __forceinline__ uint32_t tap_weight32(const Axis& a, uint32_t X, uint32_t j) {
  const int32_t d = static_cast<int32_t>((2u * j + 1u) * a.R) -
                    static_cast<int32_t>((2u * X + 1u) * a.n_in);
  const int32_t w = static_cast<int32_t>(2u * a.M) - (d < 0 ? -d : d);
  return w > 0 ? static_cast<uint32_t>(w) : 0u;
}

template <typename OutT>
__global__ void __launch_bounds__(kMmaThreads, 2) preba_antialias_mma_kernel(const Params p) {
  extern __shared__ __align__(16) uint8_t smem_b[];
  const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5, C = p.C;
  const uint32_t chunks = (C + p.mma_rows - 1) / p.mma_rows, groups = (C + kGroup - 1) / kGroup;
  const uint32_t img = blockIdx.x / (chunks * groups);
  const uint32_t rest = blockIdx.x - img * chunks * groups;
  const uint32_t k0 = (rest / groups) * p.mma_rows, xg0 = (rest % groups) * kGroup;
  const preba_img_t e = p.table[img];
  const uint64_t usable = p.pixels_bytes & ~15ull;
  if (e.h < 1 || e.w < 1 || e.h > PREBA_MAX_DIM || e.w > PREBA_MAX_DIM ||
      e.offset % PREBA_PACK_ALIGN != 0 || e.offset > usable ||
      3ull * e.h * e.w > usable - e.offset) {
    if (tid == 0 && rest == 0) report(p.status, PREBA_ERR_BAD_TABLE);
    return;
  }
  uint32_t rh, rw, top, left;
  resized_size(e.h, e.w, p.S, &rh, &rw);
  if (p.crop) {
    top = p.crop[2 * img];
    left = p.crop[2 * img + 1];
    if (static_cast<uint64_t>(top) + C > rh || static_cast<uint64_t>(left) + C > rw) {
      if (tid == 0 && rest == 0) report(p.status, PREBA_ERR_BAD_CROP);
      return;
    }
  } else {
    top = (rh - C) / 2;
    left = (rw - C) / 2;
  }
  const Axis ax = make_axis(e.w, rw), ay = make_axis(e.h, rh);
  MmaPlan pl;
  if (mm2_plan(ax, ay, e.w, C, p.mm2_smem, nullptr)) return;  // the chained kernel's image
  if (!mma_plan(ax, ay, e.w, C, p.mma_smem, &pl)) return;    // the general kernel's image

  float* hbuf = reinterpret_cast<float*>(smem_b + pl.off_h);
  uint16_t* wxi = reinterpret_cast<uint16_t*>(smem_b + pl.off_wx);
  uint32_t* xlo = reinterpret_cast<uint32_t*>(smem_b + pl.off_xlo);
  uint32_t* xcnt = reinterpret_cast<uint32_t*>(smem_b + pl.off_xcnt);
  float* invx = reinterpret_cast<float*>(smem_b + pl.off_invx);
  float* wyn = reinterpret_cast<float*>(smem_b + pl.off_wy);
  uint32_t* ylo = reinterpret_cast<uint32_t*>(smem_b + pl.off_ylo);
  uint32_t* ycnt = reinterpret_cast<uint32_t*>(smem_b + pl.off_ycnt);
  const uint32_t bars = smem_addr(smem_b + pl.off_bar);
  const uint8_t* ring_p = smem_b + pl.off_ring;
  const uint32_t ring = smem_addr(ring_p);
  const uint32_t ncols = C - xg0 < kGroup ? C - xg0 : kGroup;
  const uint32_t nrows = C - k0 < p.mma_rows ? C - k0 : p.mma_rows;

  // tables: a thread per row of the CTA, and per column of the group
  if (tid < nrows) {
    const uint32_t Y = top + k0 + tid;
    uint32_t j0, j1;
    tap_range32(ay, Y, &j0, &j1);
    uint32_t sum = 0;
    for (uint32_t j = j0; j < j1; ++j) sum += tap_weight32(ay, Y, j);
    const float inv = 1.0f / static_cast<float>(sum);
    for (uint32_t j = j0; j < j1; ++j)
      wyn[tid * kMaxTapsY + (j - j0)] = static_cast<float>(tap_weight32(ay, Y, j)) * inv;
    ylo[tid] = j0;
    ycnt[tid] = j1 - j0;
  }
  if (tid < kGroup) {
    uint32_t j0 = 0, j1 = 0;
    float inv = 0.f;
    if (tid < ncols) {
      const uint32_t X = left + xg0 + tid;
      tap_range32(ax, X, &j0, &j1);
      uint32_t sum = 0;
      for (uint32_t j = j0; j < j1; ++j) {
        const uint32_t wgt = tap_weight32(ax, X, j);
        wxi[tid * kMaxTapsX + (j - j0)] = static_cast<uint16_t>(wgt);
        sum += wgt;
      }
      inv = 1.0f / static_cast<float>(sum);
    }
    xlo[tid] = j0;
    xcnt[tid] = j1 - j0;
    invx[tid] = inv;
  }
  if (tid == 0) {
    for (uint32_t s = 0; s < pl.slots; ++s) mbar_init(bars + 8u * s, 16);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  // the bytes of an input row under the group, and the input rows under the CTA's output rows
  const uint32_t rowbyte0 = 3u * xlo[0];
  const uint32_t rowbytes = 3u * (xlo[ncols - 1] + xcnt[ncols - 1]) - rowbyte0;
  const uint32_t ya = ylo[0], yb = ylo[nrows - 1] + ycnt[nrows - 1];
  const uint32_t ntiles16 = (yb - ya + 15u) / 16u;
  const uint8_t* image = p.pixels + e.offset;
  const uint8_t* stop = p.pixels + usable;
  const uint64_t pitch = 3ull * e.w;
  if (16u + rowbytes + kTileBytes > pl.seg) {  // cannot happen within the plan's bounds
    if (tid == 0) report(p.status, PREBA_ERR_TOO_LARGE);
    return;
  }
  // rows start on the same byte phase (the pitch is a multiple of 4)
  const uint32_t skew4 = static_cast<uint32_t>(reinterpret_cast<uintptr_t>(image + rowbyte0)) & 3u;

  // Warp 0 asks for the 16 rows of tile m, a lane per row: a row the CTA needs is copied and
  // its bytes announced to the slot's barrier, the other lanes of the sixteen just arrive.
  auto issue = [&](uint32_t m) {
    if (lane >= 16u) return;
    const uint32_t slot = m % pl.slots, bar = bars + 8u * slot;
    const uint32_t r = ya + 16u * m + lane;
    if (r < yb) {
      const uint8_t* src = image + r * pitch + rowbyte0;
      const uint32_t skew = static_cast<uint32_t>(reinterpret_cast<uintptr_t>(src)) & 15u;
      uint32_t bytes = (skew + rowbytes + 15u) & ~15u;
      if (bytes > static_cast<uint64_t>(stop - (src - skew)))  // only padding is lost
        bytes = static_cast<uint32_t>(stop - (src - skew));
      fence_async_shared();
      // checked build: the row lies in its place in the ring and in the pixel buffer
      if (PREBA_IN_RANGE(p.status, bytes <= pl.seg && src - skew >= p.pixels &&
                                       src - skew + bytes <= p.pixels + p.pixels_bytes)) {
        mbar_arrive_expect_tx(bar, bytes);
        bulk_copy_g2s(ring + (slot * 16u + lane) * pl.seg, src - skew, bytes, bar);
      } else {
        mbar_arrive(bar);
      }
    } else {
      mbar_arrive(bar);
    }
  };
  if (warp == 0)
    for (uint32_t m = 0; m < pl.slots && m < ntiles16; ++m) issue(m);

  // the weights of this warp's four tiles as B operands: for k-step s, register r, byte i the
  // row position kst + 32 s + 16 r + 4 q + i, for column g = 2 ch + xi the pixel X0 + xi
  const uint32_t g = lane >> 2, q = lane & 3u;
  uint32_t bhi[4][2][2], blo[4][2][2];
  int32_t kst[4];
#pragma unroll
  for (uint32_t t = 0; t < 4; ++t) {
    const uint32_t col0 = 2u * (4u * warp + t);  // first column of the tile in the group
    int32_t start = 0;
    if (col0 < ncols) {
      const int32_t nb = static_cast<int32_t>(3u * xlo[col0] - rowbyte0);
      start = nb - static_cast<int32_t>((static_cast<uint32_t>(nb) + skew4) & 3u);
    }
    kst[t] = start;
    const uint32_t ch = g >> 1, col = col0 + (g & 1u);
    const bool live = g < 6u && col < ncols;
    const uint32_t lo_px = live ? xlo[col] : 0u, n_px = live ? xcnt[col] : 0u;
#pragma unroll
    for (uint32_t s2 = 0; s2 < 2; ++s2)
#pragma unroll
      for (uint32_t r = 0; r < 2; ++r) {
        uint32_t hi = 0, lo = 0;
#pragma unroll
        for (uint32_t i = 0; i < 4; ++i) {
          const int32_t b = static_cast<int32_t>(rowbyte0) + start +
                            static_cast<int32_t>(32u * s2 + 16u * r + 4u * q + i);
          uint32_t wgt = 0;
          if (b >= 0) {
            const uint32_t px = static_cast<uint32_t>(b) / 3u;
            if (static_cast<uint32_t>(b) - 3u * px == ch && px >= lo_px && px - lo_px < n_px)
              wgt = wxi[col * kMaxTapsX + (px - lo_px)];
          }
          hi |= (wgt >> 8) << (8u * i);
          lo |= (wgt & 0xffu) << (8u * i);
        }
        bhi[t][s2][r] = hi;
        blo[t][s2][r] = lo;
      }
  }

  // the vertical pass's state: the warp's output rows are warp, warp + 8, ...; row number n of
  // them uses accumulator n % 4 (a row is finished before the row 32 further down begins);
  // columns lane and lane + 32 of the group, three channels
  float acc[4][3][2];
  uint32_t cur[4], cur0[4], cur1[4];  // the row of each accumulator and its taps [cur0, cur1)
#pragma unroll
  for (uint32_t a = 0; a < 4; ++a) {
    cur[a] = warp + 8u * a;
    const bool have = cur[a] < nrows;
    cur0[a] = have ? ylo[cur[a]] : 0xffffffffu;  // no row: never begins
    cur1[a] = have ? cur0[a] + ycnt[cur[a]] : 0xffffffffu;
#pragma unroll
    for (uint32_t c = 0; c < 3; ++c) acc[a][c][0] = acc[a][c][1] = 0.f;
  }
  OutT* out = static_cast<OutT*>(p.out) + static_cast<uint64_t>(img) * 3u * C * C;
  const float sx0 = lane < ncols ? invx[lane] : 0.f;
  const float sx1 = lane + 32u < ncols ? invx[lane + 32u] : 0.f;

  // horizontal pass of tile m: H = rows x weights on the tensor cores, into buffer m % 2
  auto horizontal = [&](uint32_t m) {
    const uint32_t slot = m % pl.slots, r0 = ya + 16u * m;
    float* hb = hbuf + (m & 1u) * kHFloats;
    // rows g and g + 8 of the tile: where their first needed byte lies in the slot
    const uint32_t sk0 = static_cast<uint32_t>(
        reinterpret_cast<uintptr_t>(image + (r0 + g) * pitch + rowbyte0)) & 15u;
    const uint32_t sk1 = static_cast<uint32_t>(
        reinterpret_cast<uintptr_t>(image + (r0 + g + 8u) * pitch + rowbyte0)) & 15u;
    const uint8_t* row0 = ring_p + (slot * 16u + g) * pl.seg + sk0 + 4u * q;
    const uint8_t* row1 = ring_p + (slot * 16u + g + 8u) * pl.seg + sk1 + 4u * q;
#pragma unroll
    for (uint32_t t = 0; t < 4; ++t) {
      const uint32_t tile = 4u * warp + t;
      if (2u * tile >= ncols) break;
      // checked build: the 64 bytes each of the two rows gives to this tile lie in the row's
      // place in the ring; the tile's columns lie in H
      if (!PREBA_IN_RANGE(p.status,
                          static_cast<int32_t>(sk0 + 4u * q) + kst[t] >= 0 &&
                              static_cast<int32_t>(sk1 + 4u * q) + kst[t] >= 0 &&
                              static_cast<int32_t>((sk0 > sk1 ? sk0 : sk1) + 4u * q) + kst[t] + 52 <=
                                  static_cast<int32_t>(pl.seg) &&
                              slot < pl.slots && 2u * tile + 1u < kGroup))
        continue;
      uint32_t a[2][4];
#pragma unroll
      for (uint32_t s2 = 0; s2 < 2; ++s2) {
        const uint32_t* at0 = reinterpret_cast<const uint32_t*>(row0 + kst[t] + 32 * static_cast<int32_t>(s2));
        const uint32_t* at1 = reinterpret_cast<const uint32_t*>(row1 + kst[t] + 32 * static_cast<int32_t>(s2));
        a[s2][0] = at0[0];
        a[s2][1] = at1[0];
        a[s2][2] = at0[4];
        a[s2][3] = at1[4];
      }
      int32_t d[4] = {0, 0, 0, 0};
      mma_u8(d, a[0], bhi[t][0][0], bhi[t][0][1]);
      mma_u8(d, a[1], bhi[t][1][0], bhi[t][1][1]);
#pragma unroll
      for (uint32_t i = 0; i < 4; ++i) d[i] <<= 8;
      mma_u8(d, a[0], blo[t][0][0], blo[t][0][1]);
      mma_u8(d, a[1], blo[t][1][0], blo[t][1][1]);
      if (q < 3u) {  // columns 2 q and 2 q + 1: channel q of the tile's two pixels
        float2* h0 = reinterpret_cast<float2*>(hb + g * kHPitch + q * kHPlane + 2u * tile);
        float2* h1 = reinterpret_cast<float2*>(hb + (g + 8u) * kHPitch + q * kHPlane + 2u * tile);
        *h0 = make_float2(static_cast<float>(d[0]), static_cast<float>(d[1]));
        *h1 = make_float2(static_cast<float>(d[2]), static_cast<float>(d[3]));
      }
    }
  };

  // Tile m + 1 goes through the tensor cores while tile m's H is summed vertically: one CTA-wide
  // barrier per tile, and the wait for a tile's rows comes a whole step before they are needed.
  // Only lane 0 of a warp polls the copies' barrier.
  bool failed = false;
  auto arrived = [&](uint32_t m) {
    uint32_t ok = 1u;
    if (lane == 0) ok = mbar_wait(bars + 8u * (m % pl.slots), (m / pl.slots) & 1u) ? 1u : 0u;
    return __shfl_sync(0xffffffffu, ok, 0) != 0u;
  };
  if (!arrived(0)) failed = true;
  failed = __syncthreads_or(failed) != 0;
  if (!failed) horizontal(0);
  __syncthreads();
  if (warp == 0 && !failed && pl.slots < ntiles16) issue(pl.slots);  // tile 0's rows have been read
  for (uint32_t m = 0; m < ntiles16 && !failed; ++m) {
    const uint32_t r0 = ya + 16u * m;
    if (m + 1 < ntiles16) {
      if (arrived(m + 1)) horizontal(m + 1);
      else failed = true;
    }
    // ---- vertical pass: the tile's rows under the taps of the warp's rows in progress ----
    const float* hb = hbuf + (m & 1u) * kHFloats;
#pragma unroll
    for (uint32_t a = 0; a < 4; ++a) {
      for (;;) {
        const uint32_t y0 = cur0[a], y1 = cur1[a];
        if (y0 >= r0 + 16u) break;  // begins in a later tile (or there is no row)
        const uint32_t yl = cur[a];
        const uint32_t from = y0 > r0 ? y0 : r0, to = y1 < r0 + 16u ? y1 : r0 + 16u;
        const float* wrow = wyn + yl * kMaxTapsY + (from - y0);
        const float* h = hb + (from - r0) * kHPitch + lane;
        // checked build: the taps lie in the row's weights, the rows in the tile of H, the
        // output row in the crop
        if (!PREBA_IN_RANGE(p.status, yl < kMmaRows && yl < nrows && y1 - y0 <= kMaxTapsY &&
                                          from >= r0 && to <= r0 + 16u && k0 + yl < C))
          break;
        for (uint32_t r = from; r < to; ++r, ++wrow, h += kHPitch) {
          const float wgt = *wrow;
#pragma unroll
          for (uint32_t c = 0; c < 3; ++c) {
            acc[a][c][0] = fmaf(wgt, h[c * kHPlane], acc[a][c][0]);
            acc[a][c][1] = fmaf(wgt, h[c * kHPlane + 32u], acc[a][c][1]);
          }
        }
        if (y1 > r0 + 16u) break;  // goes on in the next tile
        // the row's last tap has passed: normalise, store, on to the warp's row 32 further down
#pragma unroll
        for (uint32_t c = 0; c < 3; ++c) {
          const uint64_t at = (static_cast<uint64_t>(c) * C + (k0 + yl)) * C + xg0 + lane;
          if (lane < ncols) out[at] = to_out<OutT>(fmaf(acc[a][c][0] * sx0, p.mul[c], p.add[c]));
          if (lane + 32u < ncols)
            out[at + 32u] = to_out<OutT>(fmaf(acc[a][c][1] * sx1, p.mul[c], p.add[c]));
          acc[a][c][0] = acc[a][c][1] = 0.f;
        }
        cur[a] = yl + 32u;
        const bool have = yl + 32u < nrows;
        cur0[a] = have ? ylo[yl + 32u] : 0xffffffffu;
        cur1[a] = have ? cur0[a] + ycnt[yl + 32u] : 0xffffffffu;
      }
    }
    // tile m + 1's H is complete, tile m's has been read, and so have the staged rows of tile
    // m + 1: their slot takes the rows of tile m + 1 + slots
    failed = __syncthreads_or(failed) != 0;
    if (warp == 0 && !failed && m + 1 + pl.slots < ntiles16) issue(m + 1 + pl.slots);
  }
  if (failed && tid == 0) {
    report(p.status, PREBA_ERR_TIMEOUT);
    // copies already asked for may still be landing in the ring: wait for them (bounded)
    for (uint32_t s = 0; s < pl.slots; ++s) {
      (void)mbar_wait(bars + 8u * s, 0u);
      (void)mbar_wait(bars + 8u * s, 1u);
    }
  }
}

__device__ __forceinline__ void mma_f16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0,
                                        uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
      "{%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// Two bytes of x (bytes 0 and 1 if PAIR == 0, bytes 2 and 3 if PAIR == 1) as a pair of binary16
// numbers, each times a power of two: a byte b under the exponent byte 0x64 is the number
// 1024 + b, and one fused multiply-add, (1024 + b) * mul - 1024 * mul, leaves b * mul exactly
// (mul and off are the binary16 patterns of mul and of -1024 * mul).
__device__ __forceinline__ uint32_t scale_biased(uint32_t biased, uint32_t mul, uint32_t off) {
  uint32_t r;
  const uint32_t mul2 = mul | (mul << 16), off2 = off | (off << 16);
  asm("fma.rn.f16x2 %0, %1, %2, %3;" : "=r"(r) : "r"(biased), "r"(mul2), "r"(off2));
  return r;
}
template <uint32_t PAIR>
__device__ __forceinline__ uint32_t expand_bytes(uint32_t x, uint32_t mul, uint32_t off) {
  return scale_biased(__byte_perm(x, 0x64646464u, PAIR == 0 ? 0x4140u : 0x4342u), mul, off);
}

template <typename OutT, uint32_t KS>
__global__ void __launch_bounds__(kT2Threads, 2) preba_antialias_mm2_kernel(const Params p) {
  extern __shared__ __align__(16) uint8_t smem_b[];
  const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5, C = p.C;
  const uint32_t chunks = (C + p.mm2_rows - 1) / p.mm2_rows, groups = (C + kT2Group - 1) / kT2Group;
  const uint32_t img = blockIdx.x / (chunks * groups);
  const uint32_t rest = blockIdx.x - img * chunks * groups;
  const uint32_t k0 = (rest / groups) * p.mm2_rows, xg0 = (rest % groups) * kT2Group;
  const preba_img_t e = p.table[img];
  const uint64_t usable = p.pixels_bytes & ~15ull;
  if (e.h < 1 || e.w < 1 || e.h > PREBA_MAX_DIM || e.w > PREBA_MAX_DIM ||
      e.offset % PREBA_PACK_ALIGN != 0 || e.offset > usable ||
      3ull * e.h * e.w > usable - e.offset) {
    if (tid == 0 && rest == 0 && KS == 3u) report(p.status, PREBA_ERR_BAD_TABLE);
    return;
  }
  uint32_t rh, rw, top, left;
  resized_size(e.h, e.w, p.S, &rh, &rw);
  if (p.crop) {
    top = p.crop[2 * img];
    left = p.crop[2 * img + 1];
    if (static_cast<uint64_t>(top) + C > rh || static_cast<uint64_t>(left) + C > rw) {
      if (tid == 0 && rest == 0 && KS == 3u) report(p.status, PREBA_ERR_BAD_CROP);
      return;
    }
  } else {
    top = (rh - C) / 2;
    left = (rw - C) / 2;
  }
  const Axis ax = make_axis(e.w, rw), ay = make_axis(e.h, rh);
  Mm2Plan pl;
  if (!mm2_plan(ax, ay, e.w, C, p.mm2_smem, &pl) || pl.ks != KS) return;  // another kernel's image

  uint16_t* wxi = reinterpret_cast<uint16_t*>(smem_b + pl.off_wx);
  uint32_t* xlo = reinterpret_cast<uint32_t*>(smem_b + pl.off_xlo);
  uint32_t* xcnt = reinterpret_cast<uint32_t*>(smem_b + pl.off_xcnt);
  float* invx = reinterpret_cast<float*>(smem_b + pl.off_invx);
  uint32_t* ylo = reinterpret_cast<uint32_t*>(smem_b + pl.off_ylo);
  uint32_t* yhi = reinterpret_cast<uint32_t*>(smem_b + pl.off_yhi);
  float* invy = reinterpret_cast<float*>(smem_b + pl.off_invy);
  uint4* meta = reinterpret_cast<uint4*>(smem_b + pl.off_meta);
  const uint32_t full = smem_addr(smem_b + pl.off_bar), empty = full + 8u * kT2MaxSlots;
  const uint8_t* ring_p = smem_b + pl.off_ring;
  const uint32_t ring = smem_addr(ring_p);
  const uint32_t ncols = C - xg0 < kT2Group ? C - xg0 : kT2Group;
  const uint32_t nrows = C - k0 < p.mm2_rows ? C - k0 : p.mm2_rows;

  // tables: a thread per row of the CTA, and per column of the group
  if (tid < nrows) {
    const uint32_t Y = top + k0 + tid;
    uint32_t j0, j1;
    tap_range32(ay, Y, &j0, &j1);
    uint32_t sum = 0;
    for (uint32_t j = j0; j < j1; ++j) sum += tap_weight32(ay, Y, j);
    ylo[tid] = j0;
    yhi[tid] = j1;
    invy[tid] = 1.0f / static_cast<float>(sum);
  }
  if (tid >= 256u && tid - 256u < kT2Group) {
    const uint32_t col = tid - 256u;
    uint32_t j0 = 0, j1 = 0;
    float inv = 0.f;
    if (col < ncols) {
      const uint32_t X = left + xg0 + col;
      tap_range32(ax, X, &j0, &j1);
      uint32_t sum = 0;
      for (uint32_t j = j0; j < j1; ++j) {
        const uint32_t wgt = tap_weight32(ax, X, j);
        wxi[col * kMaxTapsX + (j - j0)] = static_cast<uint16_t>(wgt);
        sum += wgt;
      }
      inv = 1.0f / static_cast<float>(sum);
    }
    xlo[col] = j0;
    xcnt[col] = j1 - j0;
    invx[col] = inv;
  }
  if (tid == 0) {
    for (uint32_t s = 0; s < pl.slots; ++s) {
      mbar_init(full + 8u * s, 16);
      mbar_init(empty + 8u * s, kT2Tiles);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  // the bytes of an input row under the group, and the input rows under the CTA's output rows
  const uint32_t rowbyte0 = 3u * xlo[0];
  const uint32_t rowbytes = 3u * (xlo[ncols - 1] + xcnt[ncols - 1]) - rowbyte0;
  // Tiles of sixteen input rows start at multiples of 16 in the image, whatever rows the CTA
  // has: the sums of an output row are then grouped alike however the image is cut into CTAs,
  // and the result does not depend on the cut.
  const uint32_t ya_need = ylo[0], ya = ya_need & ~15u, yb = yhi[nrows - 1];
  const uint32_t ntiles16 = (yb - ya + 15u) / 16u;
  const uint32_t mtiles = (ncols + kT2Px - 1u) / kT2Px;
  const uint8_t* image = p.pixels + e.offset;
  const uint8_t* stop = p.pixels + usable;
  const uint64_t pitch = 3ull * e.w;
  // rows start on the same byte phase (the pitch is a multiple of 4)
  const uint32_t skew4 = static_cast<uint32_t>(reinterpret_cast<uintptr_t>(image + rowbyte0)) & 3u;
  const uint32_t g = lane >> 2, q = lane & 3u;

  // The window of this warp's M-tile.  Cannot happen within the plan's bounds: a row longer
  // than its place in the ring, or pixels whose taps do not fit the window; the CTA leaves as
  // one.
  const bool live = warp < mtiles;
  const uint32_t col0 = kT2Px * warp;
  int32_t kst = 0;
  bool fits = 16u + rowbytes + 32u * KS <= pl.seg;
  if (live) {
    const uint32_t c1 = col0 + kT2Px - 1u < ncols ? col0 + kT2Px - 1u : ncols - 1u;
    const uint32_t nb = 3u * xlo[col0] - rowbyte0, gap = (nb + skew4) & 3u;
    kst = static_cast<int32_t>(nb) - static_cast<int32_t>(gap);
    if (3u * (xlo[c1] + xcnt[c1]) - rowbyte0 - nb + gap > 32u * KS) fits = false;
  }
  if (!__syncthreads_and(fits)) {
    if (tid == 0) report(p.status, PREBA_ERR_TOO_LARGE);
    return;
  }

  if (warp == kT2Tiles) {
    // ---- the feeding warp ----------------------------------------------------------------------
    const int32_t two_m = static_cast<int32_t>(2u * ay.M), two_r = static_cast<int32_t>(2u * ay.R);
    uint32_t ynext = 0;  // the first output row of the CTA whose last tap has not passed
    bool failed = false;
    // (slot and use of tile m: m % slots and m / slots, counted along)
    uint32_t slot = 0, use = 0;
    for (uint32_t m = 0; m < ntiles16; ++m, slot = slot + 1u == pl.slots ? 0u : slot + 1u,
                  use += slot == 0u ? 1u : 0u) {
      const uint32_t r0 = ya + 16u * m, bar = full + 8u * slot;
      if (use > 0u) {  // every warp has given the slot back
        if (!mbar_wait_parked(empty + 8u * slot, (use - 1u) & 1u)) failed = true;
        if (__any_sync(0xffffffffu, failed)) {
          failed = true;
          break;
        }
      }
      // The weights of the output rows under this tile, as the B operand of the second
      // product (16 input rows x 8 output rows, binary16): column g is the row with
      // yl % 8 == g among ynext .. ynext + 7, the lane's k are input rows
      // r0 + {2q, 2q + 1, 8 + 2q, 9 + 2q}.  An integer weight w < 2^16 goes in as two exact
      // pieces, (w & 255) / 256 and w >> 8.
      uint4 wrec = make_uint4(0u, 0u, 0u, 0u), drec;
      {
        const uint32_t yl = ynext + ((g - ynext) & 7u);
        uint32_t w4[4] = {0u, 0u, 0u, 0u};
        if (yl < nrows) {
          const uint32_t Y = top + k0 + yl, rbase = r0 + 2u * q;
          const int32_t d = static_cast<int32_t>((2u * rbase + 1u) * ay.R) -
                            static_cast<int32_t>((2u * Y + 1u) * ay.n_in);
#pragma unroll
          for (uint32_t i = 0; i < 4; ++i) {
            const uint32_t dr = (i & 1u) + 8u * (i >> 1);
            const int32_t di = d + static_cast<int32_t>(dr) * two_r;
            int32_t wgt = two_m - (di < 0 ? -di : di);
            if (wgt < 0 || rbase + dr >= ay.n_in) wgt = 0;
            w4[i] = static_cast<uint32_t>(wgt);
          }
        }
        const uint32_t pair0 = __byte_perm(w4[0], w4[1], 0x5140);  // low, low, high, high bytes
        const uint32_t pair1 = __byte_perm(w4[2], w4[3], 0x5140);
        wrec.x = expand_bytes<0>(pair0, 0x1c00u, 0xc400u);  // (1024 + b) / 256 - 4
        wrec.y = expand_bytes<0>(pair1, 0x1c00u, 0xc400u);
        wrec.z = expand_bytes<1>(pair0, 0x3c00u, 0xe400u);  // (1024 + b) - 1024
        wrec.w = expand_bytes<1>(pair1, 0x3c00u, 0xe400u);
      }
      // rows that are complete after this tile, for the lane's two columns of the second product
      {
        const uint32_t y0 = ynext + ((2u * q - ynext) & 7u), y1 = ynext + ((2u * q + 1u - ynext) & 7u);
        const bool d0 = y0 < nrows && yhi[y0] <= r0 + 16u, d1 = y1 < nrows && yhi[y1] <= r0 + 16u;
        drec.x = d0 ? y0 : 0xffffffffu;
        drec.y = d1 ? y1 : 0xffffffffu;
        drec.z = __float_as_uint(d0 ? invy[y0] : 0.f);
        drec.w = __float_as_uint(d1 ? invy[y1] : 0.f);
      }
      meta[slot * (kT2MetaBytes / 16u) + lane] = wrec;
      meta[slot * (kT2MetaBytes / 16u) + 32u + lane] = drec;
      {
        const uint32_t yl = ynext + (lane & 7u);
        const bool done = yl < nrows && yhi[yl] <= r0 + 16u;
        const uint32_t mask = __ballot_sync(0xffffffffu, done) & 0xffu;
        ynext += static_cast<uint32_t>(__ffs(static_cast<int>(~mask))) - 1u;
      }
      __syncwarp();  // the record is written before any lane announces the tile
      // the 16 rows of the tile, a lane per row: a row the CTA needs is copied and its bytes
      // announced to the slot's barrier, the other lanes of the sixteen just arrive
      if (lane < 16u) {
        const uint32_t r = r0 + lane;
        bool copied = false;
        if (r >= ya_need && r < yb) {  // (rows before the first needed one get no weight)
          const uint8_t* src = image + r * pitch + rowbyte0;
          const uint32_t skew = static_cast<uint32_t>(reinterpret_cast<uintptr_t>(src)) & 15u;
          uint32_t bytes = (skew + rowbytes + 15u) & ~15u;
          if (bytes > static_cast<uint64_t>(stop - (src - skew)))  // only padding is lost
            bytes = static_cast<uint32_t>(stop - (src - skew));
          fence_async_shared();
          // checked build: the row lies in its place in the ring and in the pixel buffer
          if (PREBA_IN_RANGE(p.status, bytes <= pl.seg && src - skew >= p.pixels &&
                                           src - skew + bytes <= p.pixels + p.pixels_bytes)) {
            mbar_arrive_expect_tx(bar, bytes);
            bulk_copy_g2s(ring + (slot * 16u + lane) * pl.seg, src - skew, bytes, bar);
            copied = true;
          }
        }
        if (!copied) mbar_arrive(bar);
      }
    }
    if (failed) {
      if (lane == 0) report(p.status, PREBA_ERR_TIMEOUT);
      // copies already asked for may still be landing in the ring: wait for them (bounded)
      // before the CTA's shared memory is given up
      if (lane == 0)
        for (uint32_t s = 0; s < pl.slots; ++s) {
          (void)mbar_wait(full + 8u * s, 0u);
          (void)mbar_wait(full + 8u * s, 1u);
        }
    }
    return;
  }

  // ---- the warps that own an M-tile ----------------------------------------------------------------
  // The weights as A operands.  Row mr of the M-tile is channel mr % 3 of the tile's pixel
  // mr / 3 (row 15 is unused); register r holds row g (+ 8 if r is odd), bytes
  // k = 16 (r / 2) + 4 q + i of step s: the row position kst + 32 s + k.
  uint32_t ahi[KS][4], alo[KS][4];
  float scale[2];  // per row (g, g + 8): 2^22 / (sum of the column's weights * 255 std)
#pragma unroll
  for (uint32_t half = 0; half < 2; ++half) {
    const uint32_t mr = g + 8u * half, col = col0 + mr / 3u, ch = mr % 3u;
    const float mul = ch == 0u ? p.mul[0] : (ch == 1u ? p.mul[1] : p.mul[2]);
    // (the second product leaves 2^-22 times the sum)
    scale[half] = (live && mr < 15u && col < ncols) ? invx[col] * mul * 4194304.f : 0.f;
  }
  {
    // The lane's first byte of the window as pixel and channel (three bytes further on, so
    // that the number is not negative), then byte by byte: (rem + o) / 3 for o < 500 is
    // ((rem + o) * 171) >> 9.
    const uint32_t first = static_cast<uint32_t>(static_cast<int32_t>(rowbyte0) + kst +
                                                 static_cast<int32_t>(4u * q) + 3);
    const uint32_t first_px = first / 3u, first_rem = first - 3u * first_px;
#pragma unroll
    for (uint32_t r = 0; r < 4; ++r) {
      const uint32_t mr = g + 8u * (r & 1u), ch = mr % 3u, col = col0 + mr / 3u;
      const bool on = live && mr < 15u && col < ncols;
      // taps of the column as pixel numbers shifted like first_px; none if the row is unused
      const uint32_t lo_px = on ? xlo[col] + 1u : 1u, n_px = on ? xcnt[col] : 0u;
      const uint16_t* wrow = wxi + col * kMaxTapsX;
#pragma unroll
      for (uint32_t s = 0; s < KS; ++s) {
        uint32_t hi = 0, lo = 0;
#pragma unroll
        for (uint32_t i = 0; i < 4; ++i) {
          const uint32_t o = first_rem + 32u * s + 16u * (r >> 1) + i;
          const uint32_t dpx = (o * 171u) >> 9, rem = o - 3u * dpx;
          const uint32_t tap = first_px + dpx - lo_px;  // wraps below the first tap
          uint32_t wgt = 0;
          if (rem == ch && tap < n_px) wgt = wrow[tap];
          hi |= (wgt >> 8) << (8u * i);
          lo |= (wgt & 0xffu) << (8u * i);
        }
        ahi[s][r] = hi;
        alo[s][r] = lo;
      }
    }
  }
  // where the lane's two rows of the M-tile go: plane of the channel, column of the pixel
  const uint32_t px_a = g / 3u, px_b = (g + 8u) / 3u;
  const uint32_t ch_a = g % 3u, ch_b = (g + 8u) % 3u;
  const float add_a = ch_a == 0u ? p.add[0] : (ch_a == 1u ? p.add[1] : p.add[2]);
  const float add_b = ch_b == 0u ? p.add[0] : (ch_b == 1u ? p.add[1] : p.add[2]);
  OutT* out = static_cast<OutT*>(p.out) + static_cast<uint64_t>(img) * 3u * C * C;
  OutT* out_a = out + static_cast<uint64_t>(ch_a) * C * C + xg0 + col0 + px_a;
  OutT* out_b = out + static_cast<uint64_t>(ch_b) * C * C + xg0 + col0 + px_b;

  // The vertical sums: output row yl of the CTA uses column yl % 8 of the second product; a lane
  // holds columns 2q and 2q + 1 of rows g and g + 8.
  float acc[4] = {0.f, 0.f, 0.f, 0.f};
  // 16-byte skew of input row r: (base + r * pitch) & 15, in 32 bits
  const uint32_t skew_base = static_cast<uint32_t>(reinterpret_cast<uintptr_t>(image + rowbyte0)) & 15u;
  const uint32_t skew_step = static_cast<uint32_t>(pitch & 15u);
  const uint8_t* ring_row0 = ring_p + g * pl.seg + 4u * q + kst;
  const uint8_t* ring_row1 = ring_row0 + 8u * pl.seg;

  bool failed = false;
  uint32_t slot = 0, use = 0;  // of tile m: m % slots and m / slots, counted along
  for (uint32_t m = 0; m < ntiles16; ++m, slot = slot + 1u == pl.slots ? 0u : slot + 1u,
                use += slot == 0u ? 1u : 0u) {
    const uint32_t r0 = ya + 16u * m;
    if (!mbar_wait_parked(full + 8u * slot, use & 1u)) failed = true;
    if (__any_sync(0xffffffffu, failed)) {
      failed = true;
      break;
    }
    if (live) {
      const uint4 wrec = meta[slot * (kT2MetaBytes / 16u) + lane];
      const uint4 drec = meta[slot * (kT2MetaBytes / 16u) + 32u + lane];
      // rows g and g + 8 of the tile: where their first needed byte lies in the slot
      const uint32_t sk0 = (skew_base + (r0 + g) * skew_step) & 15u;
      const uint32_t sk1 = (skew_base + (r0 + g + 8u) * skew_step) & 15u;
      // checked build: the window of both rows lies in the row's place in the ring
      if (PREBA_IN_RANGE(p.status,
                         static_cast<int32_t>(sk0 + 4u * q) + kst >= 0 &&
                             static_cast<int32_t>(sk1 + 4u * q) + kst >= 0 &&
                             static_cast<int32_t>((sk0 > sk1 ? sk0 : sk1) + 4u * q) + kst +
                                     static_cast<int32_t>(32u * KS - 12u) <=
                                 static_cast<int32_t>(pl.seg) &&
                             slot < pl.slots)) {
        // first product, high and low bytes of the weights apart: e = rows 0-7 of the tile,
        // f = rows 8-15
        // (the low sums start at 0x64 in their top byte, which H never reaches: the exponent
        // byte of the binary16 pieces below comes along for free)
        constexpr int32_t kTop = 0x64000000;
        int32_t eh[4] = {0, 0, 0, 0}, el[4] = {kTop, kTop, kTop, kTop}, fh[4] = {0, 0, 0, 0},
                fl[4] = {kTop, kTop, kTop, kTop};
        const uint32_t* at0 = reinterpret_cast<const uint32_t*>(ring_row0 + slot * 16u * pl.seg + sk0);
        const uint32_t* at1 = reinterpret_cast<const uint32_t*>(ring_row1 + slot * 16u * pl.seg + sk1);
#pragma unroll
        for (uint32_t s = 0; s < KS; ++s) {
          const uint32_t b00 = at0[8 * s], b01 = at0[8 * s + 4], b10 = at1[8 * s], b11 = at1[8 * s + 4];
          mma_u8(eh, ahi[s], b00, b01);
          mma_u8(el, alo[s], b00, b01);
          mma_u8(fh, ahi[s], b10, b11);
          mma_u8(fl, alo[s], b10, b11);
        }
        // H = 256 high + low, below 2^24, under the byte 0x64; register i: row g + 8 (i / 2),
        // input row 2q + i % 2
        uint32_t he[4], hf[4];
#pragma unroll
        for (uint32_t i = 0; i < 4; ++i) {
          he[i] = (static_cast<uint32_t>(eh[i]) << 8) + static_cast<uint32_t>(el[i]);
          hf[i] = (static_cast<uint32_t>(fh[i]) << 8) + static_cast<uint32_t>(fl[i]);
        }
        // The three bytes of H as binary16 A operands of the second product (16 (x, ch) rows
        // by 16 input rows): byte 0 scaled by 2^-14, byte 1 by 2^-6, byte 2 by 4, all exact,
        // so that the sum is 2^-22 times sum_r w[r] H[r].
#pragma unroll
        for (uint32_t pln = 0; pln < 3; ++pln) {
          uint32_t a[4];
#pragma unroll
          for (uint32_t h = 0; h < 2; ++h) {
            // bytes pln of the four values of row g + 8 h: input rows 2q, 2q + 1 (e),
            // 8 + 2q, 9 + 2q (f)
            // one permute puts each byte under the exponent byte: the numbers 1024 + byte
            const uint32_t sel = pln == 0 ? 0x7430u : (pln == 1 ? 0x7531u : 0x7632u);
            const uint32_t pe = __byte_perm(he[2 * h], he[2 * h + 1], sel);
            const uint32_t pf = __byte_perm(hf[2 * h], hf[2 * h + 1], sel);
            const uint32_t mul = pln == 0 ? 0x0400u : (pln == 1 ? 0x2400u : 0x4400u);
            const uint32_t off = pln == 0 ? 0xac00u : (pln == 1 ? 0xcc00u : 0xec00u);
            a[h] = scale_biased(pe, mul, off);      // k = 2q, 2q + 1
            a[2 + h] = scale_biased(pf, mul, off);  // k = 8 + 2q, 9 + 2q
          }
          mma_f16(acc, a, wrec.x, wrec.y);
          mma_f16(acc, a, wrec.z, wrec.w);
        }
      }
      // rows whose last tap has passed: normalise, store, start the column afresh
      {
        const bool dx = drec.x != 0xffffffffu, dy = drec.y != 0xffffffffu;
        const uint32_t offx = (k0 + drec.x) * C, offy = (k0 + drec.y) * C;
        const float ix = __uint_as_float(drec.z), iy = __uint_as_float(drec.w);
        const float vx_a = fmaf(acc[0] * ix, scale[0], add_a), vx_b = fmaf(acc[2] * ix, scale[1], add_b);
        const float vy_a = fmaf(acc[1] * iy, scale[0], add_a), vy_b = fmaf(acc[3] * iy, scale[1], add_b);
        // checked build: the rows and the columns lie in the crop
        if (PREBA_IN_RANGE(p.status, (!dx || k0 + drec.x < C) && (!dy || k0 + drec.y < C) &&
                                         (scale[0] == 0.f || xg0 + col0 + px_a < C) &&
                                         (scale[1] == 0.f || xg0 + col0 + px_b < C))) {
          if (dx && scale[0] != 0.f) out_a[offx] = to_out<OutT>(vx_a);
          if (dx && scale[1] != 0.f) out_b[offx] = to_out<OutT>(vx_b);
          if (dy && scale[0] != 0.f) out_a[offy] = to_out<OutT>(vy_a);
          if (dy && scale[1] != 0.f) out_b[offy] = to_out<OutT>(vy_b);
        }
        acc[0] = dx ? 0.f : acc[0];
        acc[2] = dx ? 0.f : acc[2];
        acc[1] = dy ? 0.f : acc[1];
        acc[3] = dy ? 0.f : acc[3];
      }
    }
    // the staged rows and the record of this tile have been read: the warp gives the slot back
    __syncwarp();
    if (lane == 0) mbar_arrive(empty + 8u * slot);
  }
  if (failed && lane == 0) report(p.status, PREBA_ERR_TIMEOUT);
}

}  // namespace aa
}  // namespace preba

namespace {

using preba::aa::Params;

typedef void (*Kernel)(const Params);

Kernel kernel_for(int out_dtype) {
  return out_dtype == PREBA_F32   ? preba::aa::preba_antialias_kernel<float>
         : out_dtype == PREBA_F16 ? preba::aa::preba_antialias_kernel<__half>
                                  : preba::aa::preba_antialias_kernel<__nv_bfloat16>;
}

template <uint32_t KS>
Kernel mm2_kernel_for(int out_dtype) {
  return out_dtype == PREBA_F32   ? preba::aa::preba_antialias_mm2_kernel<float, KS>
         : out_dtype == PREBA_F16 ? preba::aa::preba_antialias_mm2_kernel<__half, KS>
                                  : preba::aa::preba_antialias_mm2_kernel<__nv_bfloat16, KS>;
}

Kernel mma_kernel_for(int out_dtype) {
  return out_dtype == PREBA_F32   ? preba::aa::preba_antialias_mma_kernel<float>
         : out_dtype == PREBA_F16 ? preba::aa::preba_antialias_mma_kernel<__half>
                                  : preba::aa::preba_antialias_mma_kernel<__nv_bfloat16>;
}

// Shared memory of the tensor-core kernel's launch: its tables, a tile of H and a ring of three
// 16-row slots of 1080p-wide groups fit, and two CTAs share an SM.
constexpr int kMmaSmemBytes = 108 * 1024;
// Of the kernel with both passes on the tensor cores, two CTAs of sixteen warps per SM: its
// tables and a ring of five 16-row slots of 1080p-wide groups.
constexpr int kMm2SmemBytes = 108 * 1024;

// Largest dynamic shared memory a CTA may ask for on the current device; the three kernels
// are opted in to it once per device.
int shared_memory_limit(cudaError_t* err) {
  constexpr int kMaxDevices = 64;
  static std::atomic<int> cache[kMaxDevices];
  int dev = -1;
  *err = cudaGetDevice(&dev);
  if (*err != cudaSuccess) return 0;
  if (dev >= 0 && dev < kMaxDevices) {
    const int known = cache[dev].load(std::memory_order_relaxed);
    if (known > 0) return known;
  }
  int optin = 0;
  *err = cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
  for (int dt : {PREBA_F32, PREBA_F16, PREBA_BF16}) {
    if (*err == cudaSuccess)
      *err = cudaFuncSetAttribute(kernel_for(dt), cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  optin);
    if (*err == cudaSuccess)
      *err = cudaFuncSetAttribute(mma_kernel_for(dt), cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  optin < kMmaSmemBytes ? optin : kMmaSmemBytes);
    if (*err == cudaSuccess)
      *err = cudaFuncSetAttribute(mm2_kernel_for<3>(dt), cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  optin < kMm2SmemBytes ? optin : kMm2SmemBytes);
    if (*err == cudaSuccess)
      *err = cudaFuncSetAttribute(mm2_kernel_for<4>(dt), cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  optin < kMm2SmemBytes ? optin : kMm2SmemBytes);
  }
  if (*err != cudaSuccess) return 0;
  if (dev >= 0 && dev < kMaxDevices) cache[dev].store(optin, std::memory_order_relaxed);
  return optin;
}

}  // namespace

extern "C" int preba_preprocess_antialias(const preba_batch_t* batch, const preba_options_t* opt,
                                          void* stream) {
  using namespace preba;
  using namespace preba::aa;
  if (!batch || !opt || !batch->pixels || !batch->table || !batch->out || batch->n == 0)
    return PREBA_ERR_INVALID_ARG;
  if (opt->flags != 0 || !dtype_ok(opt->out_dtype)) return PREBA_ERR_INVALID_ARG;
  if (batch->flags & ~PREBA_OVERLAP_PREVIOUS) return PREBA_ERR_INVALID_ARG;
  const uint32_t C = opt->out_size, S = opt->resize_short;
  if (C == 0 || S == 0 || S > PREBA_MAX_RESIZE || C > S) return PREBA_ERR_INVALID_ARG;
  for (int c = 0; c < 3; ++c)
    if (!(opt->mean[c] == opt->mean[c]) || !(opt->std[c] == opt->std[c]) || opt->std[c] == 0.f ||
        opt->std[c] - opt->std[c] != 0.f || opt->mean[c] - opt->mean[c] != 0.f)
      return PREBA_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(batch->pixels) % 16 || reinterpret_cast<uintptr_t>(batch->out) % 16 ||
      reinterpret_cast<uintptr_t>(batch->table) % 8 || reinterpret_cast<uintptr_t>(opt->crop_origin) % 4)
    return PREBA_ERR_INVALID_ARG;
  const uint64_t need = static_cast<uint64_t>(batch->n) * 3ull * C * C * dtype_bytes(opt->out_dtype);
  if (batch->out_bytes < need) return PREBA_ERR_BUFFER_TOO_SMALL;
  const uint32_t groups_at_one = C;  // CTAs of one image when every CTA makes one row
  if (static_cast<uint64_t>(batch->n) * groups_at_one > 0x7fffffffull) return PREBA_ERR_INVALID_ARG;

  cudaError_t err = cudaSuccess;
  const int limit = shared_memory_limit(&err);
  int sms = 0, dev = 0;
  if (err == cudaSuccess) err = cudaGetDevice(&dev);
  if (err == cudaSuccess) err = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (err != cudaSuccess) {
    g_last_cuda_error = static_cast<int>(err);
    return PREBA_ERR_CUDA;
  }
  // Shared memory: with the host's copy of the table, what the largest image needs; without
  // it, all a CTA may have (images that need more are reported by the kernel).
  const uint32_t limit_floats = static_cast<uint32_t>(limit) / 4u;
  uint32_t floats = limit_floats;
  const uint32_t most_rows = C + 1 < kMaxRows ? (C + 1u) & ~1u : kMaxRows;  // no CTA makes more
  // Two kernels share the batch: the tensor-core kernel takes the images mma_plan admits, the
  // other one the rest; each skips the other's images.  With the host's copy of the table a
  // kernel without images is not launched at all.
  const uint32_t mma_smem = static_cast<uint32_t>(limit < kMmaSmemBytes ? limit : kMmaSmemBytes);
  const uint32_t mm2_smem = static_cast<uint32_t>(limit < kMm2SmemBytes ? limit : kMm2SmemBytes);
  bool any_mma = true, any_rest = true, any_mm2[2] = {true, true};  // windows of 3 and 4 steps
  if (batch->table_host) {
    uint64_t most = 0;
    any_mma = any_rest = any_mm2[0] = any_mm2[1] = false;
    for (uint32_t i = 0; i < batch->n; ++i) {
      const preba_img_t& e = batch->table_host[i];
      // as in the kernel: rows are fetched in 16-byte units, so the buffer counts up to its
      // last whole unit
      const uint64_t usable = batch->pixels_bytes & ~15ull;
      if (!dims_ok(e.h, e.w) || e.offset % PREBA_PACK_ALIGN || e.offset > usable ||
          3ull * e.h * e.w > usable - e.offset)
        return PREBA_ERR_BAD_TABLE;
      uint32_t rh, rw;
      resized_size(e.h, e.w, S, &rh, &rw);
      if (opt->crop_origin_host &&
          (opt->crop_origin_host[2 * i] + static_cast<uint64_t>(C) > rh ||
           opt->crop_origin_host[2 * i + 1] + static_cast<uint64_t>(C) > rw))
        return PREBA_ERR_BAD_CROP;
      preba::aa::Mm2Plan two;
      if (mm2_plan(make_axis(e.w, rw), make_axis(e.h, rh), e.w, C, mm2_smem, &two)) {
        any_mm2[two.ks - 3u] = true;
        continue;
      }
      if (mma_plan(make_axis(e.w, rw), make_axis(e.h, rh), e.w, C, mma_smem, nullptr)) {
        any_mma = true;
        continue;
      }
      any_rest = true;
      const Plan pl = make_plan(make_axis(e.w, rw), make_axis(e.h, rh), C, most_rows);
      if (pl.off_ring > limit_floats) return PREBA_ERR_TOO_LARGE;
      // with a ring of staged rows (one pair's rows and half as many again in flight) when
      // at least the pair's rows fit, else without
      uint64_t want = pl.off_ring;
      if (plan_floats(pl, pl.tp) <= limit_floats) want = plan_floats(pl, pl.tp + pl.tp / 2 + 2);
      if (want > most) most = want;
    }
    if (most < floats) floats = static_cast<uint32_t>(most);
    if (!any_rest) floats = 0;
  }
  // Rows per CTA: the CTAs of one image are cut so that the batch fills a whole number of
  // rounds of the CTAs the GPU holds at once (a round more than needed would run nearly
  // empty), with an even number of rows (rows are made in pairs), at most kMaxRows, per CTA.
  int per_sm = 0;
  err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel_for(opt->out_dtype),
                                                      kThreads, floats * 4ull);
  if (err != cudaSuccess || per_sm < 1) {
    g_last_cuda_error = static_cast<int>(err);
    return PREBA_ERR_CUDA;
  }
  const uint64_t slots = static_cast<uint64_t>(per_sm) * sms;
  uint32_t rows = kMaxRows;
  for (uint64_t rounds = 1;; ++rounds) {
    const uint64_t per_image = rounds * slots / batch->n;
    if (per_image == 0) continue;
    rows = per_image >= C ? 1u : static_cast<uint32_t>((C + per_image - 1) / per_image);
    rows = (rows + 1u) & ~1u;
    if (rows <= most_rows) break;
  }

  Params p = {};
  p.pixels = batch->pixels;
  p.pixels_bytes = batch->pixels_bytes;
  p.table = batch->table;
  p.crop = opt->crop_origin;
  p.out = batch->out;
  p.status = batch->status;
  p.n = batch->n;
  p.C = C;
  p.S = S;
  p.rows = rows;
  p.smem_floats = floats;
  p.mma_smem = any_mma ? mma_smem : 0u;
  p.mm2_smem = (any_mm2[0] || any_mm2[1]) ? mm2_smem : 0u;
  // Output rows per CTA of the chained kernel: the chunking of an image's rows whose CTAs fill
  // the rounds of what the GPU holds at once (two CTAs per SM) best, fewest chunks first; no
  // CTA below 32 rows.
  {
    const uint64_t groups = (C + preba::aa::kT2Group - 1) / preba::aa::kT2Group;
    const uint64_t slots = 2ull * sms, least = (C + kMmaRows - 1) / kMmaRows;
    const uint64_t most_chunks = C >= 64u ? C / 32u : 1u;
    uint64_t best = least > most_chunks ? least : 0, best_fill = 0;
    for (uint64_t c = least; c <= most_chunks && c <= least + 15u; ++c) {
      const uint64_t ctas = static_cast<uint64_t>(batch->n) * groups * c;
      const uint64_t rounds = (ctas + slots - 1) / slots;
      const uint64_t fill = ctas * 1000u / (rounds * slots);
      if (fill > best_fill + 20u) best = c, best_fill = fill;  // a later choice must be clearly better
    }
    if (best == 0) best = least;
    p.mm2_rows = static_cast<uint32_t>((C + best - 1) / best);
    if (p.mm2_rows > kMmaRows) p.mm2_rows = kMmaRows;
  }
  // Output rows per CTA of the tensor-core kernel: a CTA builds its weight operands once and
  // then sweeps, so it takes as many rows as it can (all of them up to kMmaRows) unless the
  // batch then has fewer CTAs than the GPU holds at once.
  {
    const uint64_t groups = (C + kGroup - 1) / kGroup;
    const uint64_t room = 2ull * sms / (static_cast<uint64_t>(batch->n) * groups);  // chunks that fit at once
    uint64_t chunks = (C + kMmaRows - 1) / kMmaRows;
    if (room > chunks) chunks = room;
    const uint64_t most_chunks = (C + 31u) / 32u;  // no CTA below 32 rows
    if (chunks > most_chunks) chunks = most_chunks;
    uint32_t r = static_cast<uint32_t>((C + chunks - 1) / chunks);
    r = (r + 7u) & ~7u;
    p.mma_rows = r > kMmaRows ? kMmaRows : r;
  }
  for (int c = 0; c < 3; ++c) {
    p.mul[c] = static_cast<float>(1.0 / (255.0 * static_cast<double>(opt->std[c])));
    p.add[c] = static_cast<float>(-static_cast<double>(opt->mean[c]) /
                                  static_cast<double>(opt->std[c]));
  }
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  for (uint32_t v = 0; v < 2 && err == cudaSuccess; ++v) {
    if (!any_mm2[v]) continue;
    const uint64_t ctas = static_cast<uint64_t>(batch->n) * ((C + p.mm2_rows - 1) / p.mm2_rows) *
                          ((C + preba::aa::kT2Group - 1) / preba::aa::kT2Group);
    if (ctas > 0x7fffffffull) return PREBA_ERR_INVALID_ARG;
    (v == 0 ? mm2_kernel_for<3>(opt->out_dtype) : mm2_kernel_for<4>(opt->out_dtype))
        <<<static_cast<uint32_t>(ctas), preba::aa::kT2Threads, mm2_smem, s>>>(p);
    err = cudaGetLastError();
  }
  if (any_mma && err == cudaSuccess) {
    const uint64_t ctas = static_cast<uint64_t>(batch->n) * ((C + p.mma_rows - 1) / p.mma_rows) *
                          ((C + kGroup - 1) / kGroup);
    if (ctas > 0x7fffffffull) return PREBA_ERR_INVALID_ARG;
    mma_kernel_for(opt->out_dtype)<<<static_cast<uint32_t>(ctas), kMmaThreads, mma_smem, s>>>(p);
    err = cudaGetLastError();
  }
  if (any_rest && err == cudaSuccess) {
    const uint32_t grid = batch->n * ((C + rows - 1) / rows);
    kernel_for(opt->out_dtype)<<<grid, kThreads, floats * 4u, s>>>(p);
    err = cudaGetLastError();
  }
  if (err != cudaSuccess) {
    g_last_cuda_error = static_cast<int>(err);
    return PREBA_ERR_CUDA;
  }
  return PREBA_OK;
}
