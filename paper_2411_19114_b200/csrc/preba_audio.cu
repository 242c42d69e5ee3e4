// Audio path: log Mel spectrogram and per-utterance normalisation of a ragged batch (sm_100a).
//
// Kernel 1 (persistent grid): the frame pairs of the whole batch (two consecutive frames of one
// utterance) are split evenly over all resident warps, each warp taking a contiguous run.  Per
// pair the warp multiplies the two frames by the Hann window, packs them as the real and
// imaginary part of one complex sequence and runs a 512-point FFT as three passes of radix-8
// butterflies in registers, exchanging through its own shared memory between passes; window
// values and the second pass's twiddle factors are per-lane constants held in registers.  The two spectra are
// separated with one shuffle per value (the partner of bin k, bin 512 - k, sits in lane
// 32 - lane), the power spectra go to shared memory in natural order, and the triangular Mel
// filters are summed a lane per filter over a plan laid out so that no access conflicts: the
// weights iteration-major, and the filters of a half-warp starting at distinct addresses
// modulo 16.  log(energy + 2^-24) is written; frames past an utterance's own count are
// written as 0, so the result tensor needs no clearing.
// Kernel 2 (Normalize): a warp per (utterance, filter) row makes the paper's three passes over
// the row held in registers: mean, variance from that mean, normalisation.  It is launched as
// a programmatic dependent of kernel 1 and waits for it on the device.
// fp32 throughout; the path is bound by arithmetic and shared memory, not by HBM.
#include <cuda_runtime.h>

#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstdint>
#include <cstring>

#include "preba.h"
#include "preba_internal.h"

namespace preba {
namespace audio {

constexpr uint32_t kWin = PREBA_AUDIO_WIN;
constexpr uint32_t kHop = PREBA_AUDIO_HOP;
constexpr uint32_t kFft = PREBA_AUDIO_NFFT;
constexpr uint32_t kBins = kFft / 2 + 1;
constexpr uint32_t kMels = PREBA_AUDIO_MELS;
constexpr int kWarps = 4;            // warps per CTA of the spectrogram kernel
constexpr int kCtasPerSm = 3;
constexpr float kLogGuard = 5.9604644775390625e-08f;  // 2^-24
constexpr float kStdGuard = 1e-5f;

// The Mel filters as the kernel sums them.  Filter j has non-zero weight on the consecutive
// bins first[j] .. first[j] + count[j] - 1.  The 80 filters are dealt out, heaviest first, to
// five half-warps of 16 lanes over three rounds (round r: lanes 0-15 the 2r-th sixteen,
// lanes 16-31 the next).  In a round every lane reads, iteration by iteration, one weight and
// the power of one bin, starting at bin begin <= first; begin is moved down from first until
// its remainder modulo 16 is free within the half-warp, so that the 16 lanes always read 16
// different banks; the weights before first are 0.  w holds the weights iteration-major, lane
// by lane (consecutive lanes, consecutive words).
constexpr uint32_t kMelRounds = 3;
// Iterations of the three rounds as the kernel runs them (its loops are unrolled in full): the
// plan of the 80 filters at 16 kHz needs 17, 13 and 5; a round that needs fewer reads weights
// of 0, and a plan that needed more would be refused.
constexpr uint32_t kMelIters0 = 18, kMelIters1 = 14, kMelIters2 = 6;
constexpr uint32_t kMelMaxIters = kMelIters0 + kMelIters1 + kMelIters2;
constexpr uint32_t kPowPad = 16;       // zeroed entries in front of the power spectrum (begin may
                                       // lie before bin 0)
constexpr uint32_t kPowLen = kPowPad + kBins + 47;  // and behind it (rounds read past a filter's end)
struct MelPlan {
  float w[kMelMaxIters * 32];
  int16_t begin[kMelRounds][32];   // first index read in the padded power array
  uint8_t filter[kMelRounds][32];  // the lane's filter in the round, or 0xff
  uint8_t iters[kMelRounds];       // iterations the round needs (the kernel runs kMelIters*)
  uint8_t ok;                      // the plan fits the kernel's rounds and the padding
};
static_assert(sizeof(MelPlan) % 4 == 0 && sizeof(MelPlan) < 8192, "passed as a kernel parameter");

uint32_t frames_of(uint32_t length) { return length < kWin ? 0u : 1u + (length - kWin) / kHop; }

// Corner frequencies equally spaced on the HTK mel scale between 0 and rate / 2 (double);
// filter j rises from corner j to corner j + 1 and falls to corner j + 2.
MelPlan make_mel_plan() {
  MelPlan t;
  std::memset(&t, 0, sizeof(t));
  std::memset(t.filter, 0xff, sizeof(t.filter));
  const double top = 2595.0 * std::log10(1.0 + (PREBA_AUDIO_RATE / 2.0) / 700.0);
  double corner[kMels + 2];
  for (uint32_t i = 0; i < kMels + 2; ++i)
    corner[i] = 700.0 * (std::pow(10.0, (top * i / (kMels + 1)) / 2595.0) - 1.0);
  corner[0] = 0.0;
  corner[kMels + 1] = PREBA_AUDIO_RATE / 2.0;
  static float weight[kMels][kBins];
  int first[kMels], count[kMels];
  for (uint32_t j = 0; j < kMels; ++j) {
    const double lo = corner[j], mid = corner[j + 1], hi = corner[j + 2];
    first[j] = -1;
    count[j] = 0;
    for (uint32_t k = 0; k < kBins; ++k) {
      const double f = static_cast<double>(k) * PREBA_AUDIO_RATE / kFft;
      weight[j][k] = 0.f;
      if (f <= lo || f >= hi) continue;  // weight 0 at and beyond the feet
      const double wgt = f < mid ? (f - lo) / (mid - lo) : (hi - f) / (hi - mid);
      weight[j][k] = static_cast<float>(wgt);
      if (first[j] < 0) first[j] = static_cast<int>(k);
      count[j] = static_cast<int>(k) + 1 - first[j];
    }
    if (first[j] < 0) first[j] = 0;  // a filter without a bin: all weights 0
  }
  int order[kMels];
  for (uint32_t j = 0; j < kMels; ++j) order[j] = static_cast<int>(j);
  std::stable_sort(order, order + kMels, [&](int a, int b) { return count[a] > count[b]; });
  uint32_t at = 0;  // iterations used so far
  bool ok = true;
  for (uint32_t r = 0; r < kMelRounds; ++r) {
    int begin[32], filt[32];
    int iters = 0;
    for (int lane = 0; lane < 32; ++lane) begin[lane] = 0, filt[lane] = -1;
    for (int half = 0; half < 2; ++half) {
      bool used[16] = {};
      for (int i = 0; i < 16; ++i) {
        const uint32_t idx = (2 * r + half) * 16 + i;
        if (idx >= kMels) break;
        const int j = order[idx], lane = 16 * half + i;
        int e = first[j];
        while (used[((e % 16) + 16) % 16]) --e;
        used[((e % 16) + 16) % 16] = true;
        begin[lane] = e;
        filt[lane] = j;
        iters = std::max(iters, first[j] - e + count[j]);
        if (e < -static_cast<int>(kPowPad)) ok = false;
      }
    }
    const int room = static_cast<int>(r == 0 ? kMelIters0 : r == 1 ? kMelIters1 : kMelIters2);
    if (iters > room) {
      ok = false;
      break;
    }
    for (int lane = 0; lane < 32; ++lane) {
      t.begin[r][lane] = static_cast<int16_t>(begin[lane] + static_cast<int>(kPowPad));
      t.filter[r][lane] = static_cast<uint8_t>(filt[lane] < 0 ? 0xff : filt[lane]);
      if (begin[lane] + static_cast<int>(kPowPad) + room > static_cast<int>(kPowLen)) ok = false;
      for (int i = 0; i < iters; ++i) {
        const int k = begin[lane] + i;
        // a quarter of the weight: the kernel's power spectra are those of twice the spectrum
        t.w[(at + i) * 32 + lane] =
            (filt[lane] >= 0 && k >= 0 && k < static_cast<int>(kBins)) ? 0.25f * weight[filt[lane]][k]
                                                                      : 0.f;
      }
    }
    t.iters[r] = static_cast<uint8_t>(iters);
    at += room;  // the round's weights beyond `iters` stay 0
  }
  t.ok = ok ? 1 : 0;
  return t;
}

struct AudioParams {
  const float* samples;
  uint64_t samples_count;
  const preba_utt_t* table;
  float* out;
  int32_t* status;
  uint32_t n;
  uint32_t t_max;
};

__device__ __forceinline__ bool utt_ok(const preba_utt_t& u, uint64_t samples_count) {
  if (u.offset % PREBA_AUDIO_ALIGN || u.length > PREBA_AUDIO_MAX_SAMPLES) return false;
  if (u.offset > samples_count || u.length > samples_count - u.offset) return false;
  const uint32_t frames = u.length < kWin ? 0u : 1u + (u.length - kWin) / kHop;
  return u.frames == frames;
}

// Frames of utterance i that the result holds (0 for an entry that is refused).
__device__ __forceinline__ uint32_t frames_in(const AudioParams& p, uint32_t i) {
  const preba_utt_t u = p.table[i];
  return utt_ok(u, p.samples_count) ? min(u.frames, p.t_max) : 0u;
}

// The 512-point FFT runs as three passes of radix-8 butterflies held in registers
// (512 = 8 * 8 * 8).  With n = 64 n2 + 8 n1 + n0 and k = k0 + 8 k1 + 64 k2:
//   X[k] = sum_n0 W8^(n0 k2) W64^(n0 k1)
//          sum_n1 W8^(n1 k1) W512^((8 n1 + n0) k0) sum_n2 W8^(n2 k0) x[n].
// Between passes the warp exchanges its values through an 8-row array in shared memory; the
// rows are 72 elements apart after pass 1 and 66 after pass 2, which makes the 16 lanes of a
// half-warp hit 16 different 8-byte banks in every store and load.
constexpr uint32_t kPitch1 = 72;
constexpr uint32_t kPitch2 = 66;

struct __align__(16) WarpFft {
  float2 z[8 * kPitch1];   // exchange array
  float2 power[kPowLen];   // the two frames' power spectra side by side, zero padding around
};

__device__ __forceinline__ float2 cadd(float2 a, float2 b) { return make_float2(a.x + b.x, a.y + b.y); }
__device__ __forceinline__ float2 csub(float2 a, float2 b) { return make_float2(a.x - b.x, a.y - b.y); }
__device__ __forceinline__ float2 cmul(float2 a, float2 b) {
  return make_float2(a.x * b.x - a.y * b.y, a.x * b.y + a.y * b.x);
}
__device__ __forceinline__ float2 mul_neg_i(float2 a) { return make_float2(a.y, -a.x); }

// 8-point DFT in place, X[k] = sum_n v[n] exp(-2 pi i n k / 8), natural order in and out.
__device__ __forceinline__ void fft8(float2 (&v)[8]) {
  const float h = 0.70710678118654752440f;
  const float2 s0 = cadd(v[0], v[4]), s1 = cadd(v[1], v[5]), s2 = cadd(v[2], v[6]),
               s3 = cadd(v[3], v[7]);
  const float2 t0 = csub(v[0], v[4]), t1 = csub(v[1], v[5]), t2 = csub(v[2], v[6]),
               t3 = csub(v[3], v[7]);
  const float2 d0 = t0;
  const float2 d1 = make_float2(h * (t1.x + t1.y), h * (t1.y - t1.x));   // * exp(-i pi/4)
  const float2 d2 = mul_neg_i(t2);                                      // * exp(-i pi/2)
  const float2 d3 = make_float2(h * (t3.y - t3.x), -h * (t3.x + t3.y));  // * exp(-3i pi/4)
  const float2 e0 = cadd(s0, s2), e1 = csub(s0, s2), e2 = cadd(s1, s3),
               e3 = mul_neg_i(csub(s1, s3));
  const float2 o0 = cadd(d0, d2), o1 = csub(d0, d2), o2 = cadd(d1, d3),
               o3 = mul_neg_i(csub(d1, d3));
  v[0] = cadd(e0, e2);
  v[4] = csub(e0, e2);
  v[2] = cadd(e1, e3);
  v[6] = csub(e1, e3);
  v[1] = cadd(o0, o2);
  v[5] = csub(o0, o2);
  v[3] = cadd(o1, o3);
  v[7] = csub(o1, o3);
}

// One round of the Mel filters: the lane's filter summed over ITERS consecutive bins of both
// frames (weights of 0 outside the filter), then the logs.  The energies are at least 2^-24,
// a normal number, and the results lie between -17 and about 30: there the fast logarithm
// (log2 by the special-function unit times ln 2) is within 3 ulp, 6e-6 at most.
template <uint32_t ITERS>
__device__ __forceinline__ void mel_round(const float* __restrict__ wp, const float2* __restrict__ pp,
                                          uint32_t filter, float* __restrict__ out, uint32_t t_max,
                                          uint32_t t0, bool have1) {
  float e0 = 0.f, e1 = 0.f;
#pragma unroll
  for (uint32_t i = 0; i < ITERS; ++i) {
    const float wgt = wp[i * 32];
    const float2 pw = pp[i];
    e0 = fmaf(wgt, pw.x, e0);
    e1 = fmaf(wgt, pw.y, e1);
  }
  // (checked build: the caller has tested filter < 80 and t0 + 1 < t_max or the lone frame)
  if (filter != 0xffu) {
    float* __restrict__ o = out + static_cast<size_t>(filter) * t_max + t0;
    o[0] = __logf(e0 + kLogGuard);
    if (have1) o[1] = __logf(e1 + kLogGuard);
  }
}

// Frame pairs of utterance i: two frames share one complex transform.
__device__ __forceinline__ uint32_t pairs_in(const AudioParams& p, uint32_t i) {
  return (frames_in(p, i) + 1) / 2;
}

__global__ void __launch_bounds__(32 * kWarps, kCtasPerSm)
logmel_kernel(const AudioParams p, const MelPlan plan_param) {
  __shared__ WarpFft sm[kWarps];
  __shared__ float2 tw1[7][64];     // after pass 1: exp(-2 pi i col k0 / 512), k0 = 1..7, by column
  __shared__ float window[kFft];    // Hann over the first 400, then 0
  __shared__ MelPlan plan;          // lanes read different entries: shared memory, not the constant bank
  // the Normalize kernel may be scheduled as soon as resources free up; it waits for this
  // grid to complete before it reads anything
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (uint32_t k = threadIdx.x; k < kFft; k += blockDim.x) {
    window[k] = k < kWin ? 0.5f - 0.5f * cospif(2.0f * static_cast<float>(k) / kWin) : 0.f;
    if (k < 7 * 64) {
      const uint32_t k0 = (k >> 6) + 1, col = k & 63;
      float sn, cs;
      sincospif(-2.0f * static_cast<float>(col * k0) / kFft, &sn, &cs);
      tw1[k0 - 1][col] = make_float2(cs, sn);
    }
  }
  {
    const uint32_t* src = reinterpret_cast<const uint32_t*>(&plan_param);
    uint32_t* dst = reinterpret_cast<uint32_t*>(&plan);
    for (uint32_t i = threadIdx.x; i < sizeof(MelPlan) / 4; i += blockDim.x) dst[i] = src[i];
  }
  WarpFft& ws = sm[warp];
  for (uint32_t i = lane; i < kPowLen; i += 32) ws.power[i] = make_float2(0.f, 0.f);
  __syncthreads();

  // per-lane constants: the window at the lane's 13 sample positions inside the frame (of
  // 64 n2 + lane + 32 c only n2 < 6, and n2 = 6 with c = 0 and lane < 16, lie below 400), the
  // twiddles of its two columns after pass 1 and those after pass 2, its place in the Mel rounds
  const uint32_t n0 = lane & 7;
  float win[2][6], win6;
  float2 tw2[7];  // after pass 2: exp(-2 pi i n0 k1 / 64)
#pragma unroll
  for (int c = 0; c < 2; ++c)
#pragma unroll
    for (uint32_t n2 = 0; n2 < 6; ++n2) win[c][n2] = window[64 * n2 + lane + 32 * c];
  win6 = window[384 + lane];  // 0 from lane 16 on
#pragma unroll
  for (uint32_t k1 = 1; k1 < 8; ++k1) {
    float sn, cs;
    sincospif(-2.0f * static_cast<float>(n0 * k1) / 64.0f, &sn, &cs);
    tw2[k1 - 1] = make_float2(cs, sn);
  }
  float2 tw1r[2][7];  // after pass 1: the lane's two columns
#pragma unroll
  for (int c = 0; c < 2; ++c)
#pragma unroll
    for (uint32_t k0 = 1; k0 < 8; ++k0) tw1r[c][k0 - 1] = tw1[k0 - 1][lane + 32 * c];
  int mel_begin[kMelRounds];
  uint32_t mel_filter[kMelRounds];
#pragma unroll
  for (uint32_t r = 0; r < kMelRounds; ++r) {
    mel_begin[r] = plan.begin[r][lane];
    mel_filter[r] = plan.filter[r][lane];
  }

  // this warp's run of the batch's frame pairs: an equal share, contiguous
  const uint32_t nwarps = gridDim.x * kWarps, gwarp = blockIdx.x * kWarps + warp;
  uint64_t total = 0;
  for (uint32_t i0 = 0; i0 < p.n; i0 += 32) {
    uint32_t c = i0 + lane < p.n ? pairs_in(p, i0 + lane) : 0u;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
    total += c;
  }
  uint64_t g = total * gwarp / nwarps;
  const uint64_t g_end = total * (gwarp + 1) / nwarps;
  // the utterance holding pair g, and g's index in it
  uint32_t utt = 0, q = 0, upairs = 0;
  {
    uint64_t before = 0;
    bool found = false;
    for (uint32_t i0 = 0; i0 < p.n && !found; i0 += 32) {
      const uint32_t c = i0 + lane < p.n ? pairs_in(p, i0 + lane) : 0u;
      uint32_t inc = c;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t v = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= static_cast<uint32_t>(o)) inc += v;
      }
      const uint32_t hit = __ballot_sync(0xffffffffu, before + inc > g);
      if (hit) {
        const int src = __ffs(hit) - 1;
        const uint32_t inc_s = __shfl_sync(0xffffffffu, inc, src);
        upairs = __shfl_sync(0xffffffffu, c, src);
        utt = i0 + src;
        q = static_cast<uint32_t>(g - (before + inc_s - upairs));
        found = true;
      }
      before += __shfl_sync(0xffffffffu, inc, 31);
    }
    if (!found) g = g_end;  // nothing left for this warp
  }

  // The samples of a pair are fetched one pair ahead, into registers the transform has just
  // released.  The two frames overlap (the second starts 160 = 5 * 32 samples after the first),
  // so the pair is one window of 18 slots of 32 samples: slot[k] is sample 32 k + lane of the
  // first frame, which uses slots 0..12, and the second frame's slot j is slot j + 5.  Samples
  // the frames do not hold (slot 12 from lane 16 on without a second frame, slot 17 from lane
  // 16 on, slots 13..17 without a second frame) are replaced by ones that exist; they meet a
  // window weight of 0 or belong to the duplicate frame whose spectrum is not written.
  float slot[18];
  uint32_t frames = 0;
  auto fetch = [&]() {
    const preba_utt_t u = p.table[utt];
    frames = min(u.frames, p.t_max);
    const bool two = 2 * q + 1 < frames;
    const float* __restrict__ x0 = p.samples + u.offset + static_cast<size_t>(2 * q) * kHop;
    // checked build: both frames lie in the utterance and the utterance in the sample buffer
    if (!PREBA_IN_RANGE(p.status,
                        utt < p.n && 2 * q < frames &&
                            static_cast<uint64_t>(2 * q + (two ? 1 : 0)) * kHop + kWin <= u.length &&
                            u.offset + u.length <= p.samples_count)) {
#pragma unroll
      for (int k = 0; k < 18; ++k) slot[k] = 0.f;
      return;
    }
#pragma unroll
    for (uint32_t k = 0; k < 12; ++k) slot[k] = x0[32 * k + lane];
    slot[12] = x0[(two || lane < 16) ? 384 + lane : lane];
#pragma unroll
    for (uint32_t k = 13; k < 17; ++k) slot[k] = x0[two ? 32 * k + lane : 32 * (k - 13) + lane];
    slot[17] = x0[(two && lane < 16) ? 544 + lane : lane];
  };
  if (g < g_end) fetch();

#pragma unroll 1
  while (g < g_end) {
    const uint32_t t0 = 2 * q;
    const bool have1 = t0 + 1 < frames;
    float* __restrict__ out = p.out + static_cast<size_t>(utt) * kMels * p.t_max;
    // Pass 1 (over n2): a lane takes the columns 8 n1 + n0 = lane and lane + 32 of the two
    // windowed frames (real and imaginary part); the samples from 400 on are zero padding.
    float2 v[2][8];
#pragma unroll
    for (int c = 0; c < 2; ++c) {
      const uint32_t pcol = lane + 32 * c;
#pragma unroll
      for (uint32_t n2 = 0; n2 < 6; ++n2)
        v[c][n2] = make_float2(slot[2 * n2 + c] * win[c][n2], slot[2 * n2 + c + 5] * win[c][n2]);
      v[c][6] = c == 0 ? make_float2(slot[12] * win6, slot[17] * win6) : make_float2(0.f, 0.f);
      v[c][7] = make_float2(0.f, 0.f);
      fft8(v[c]);
      ws.z[pcol] = v[c][0];
#pragma unroll
      for (uint32_t k0 = 1; k0 < 8; ++k0) ws.z[k0 * kPitch1 + pcol] = cmul(v[c][k0], tw1r[c][k0 - 1]);
    }
    __syncwarp();
    // Pass 2 (over n1): a lane takes k0 = (lane + 32 c) / 8 and n0 = lane % 8.
#pragma unroll
    for (int c = 0; c < 2; ++c) {
      const uint32_t k0 = (lane >> 3) + 4 * c;
#pragma unroll
      for (uint32_t n1 = 0; n1 < 8; ++n1) v[c][n1] = ws.z[k0 * kPitch1 + 8 * n1 + n0];
    }
    __syncwarp();
#pragma unroll
    for (int c = 0; c < 2; ++c) {
      const uint32_t k0 = (lane >> 3) + 4 * c;
      fft8(v[c]);
      ws.z[n0 * kPitch2 + k0] = v[c][0];
#pragma unroll
      for (uint32_t k1 = 1; k1 < 8; ++k1)
        ws.z[n0 * kPitch2 + k0 + 8 * k1] = cmul(v[c][k1], tw2[k1 - 1]);
    }
    __syncwarp();
    // Pass 3 (over n0): a lane takes r = k0 + 8 k1 = lane + 32 c and produces Z[r + 64 k2].
#pragma unroll
    for (int c = 0; c < 2; ++c) {
      const uint32_t r = lane + 32 * c;
#pragma unroll
      for (uint32_t m = 0; m < 8; ++m) v[c][m] = ws.z[m * kPitch2 + r];
      fft8(v[c]);
    }
    // Z = A + iB with A, B the spectra of the two real frames:
    // 2 A[k] = Z[k] + conj(Z[N-k]), 2i B[k] = Z[k] - conj(Z[N-k]); the factor 1/4 of the
    // powers sits in the Mel weights.  For k = lane + 32 c + 64 k2 below 256, Z[N-k] is the
    // value (1 - c, 7 - k2) of lane 32 - lane; lane 0 finds it among its own values.
    const uint32_t partner = (32u - lane) & 31u;
#pragma unroll
    for (int c = 0; c < 2; ++c) {
#pragma unroll
      for (int k2 = 0; k2 < 4; ++k2) {
        const float2 zk = v[c][k2];
        const float2 give = v[1 - c][7 - k2];
        float2 zn = make_float2(__shfl_sync(0xffffffffu, give.x, partner),
                                __shfl_sync(0xffffffffu, give.y, partner));
        if (lane == 0) zn = c == 0 ? v[0][(8 - k2) & 7] : v[1][7 - k2];
        const float ar = zk.x + zn.x, ai = zk.y - zn.y;
        const float br = zk.y + zn.y, bi = zn.x - zk.x;
        ws.power[kPowPad + lane + 32 * c + 64 * k2] =
            make_float2(ar * ar + ai * ai, br * br + bi * bi);
      }
    }
    if (lane == 0) {  // bin 256 is its own partner
      const float ar = 2.f * v[0][4].x, br = 2.f * v[0][4].y;
      ws.power[kPowPad + 256] = make_float2(ar * ar, br * br);
    }
    __syncwarp();
    // on to the next pair that has frames; its samples travel while the filters are summed
    const uint32_t this_t0 = t0;
    ++g;
    ++q;
    if (g < g_end) {
      while (q >= upairs) {
        ++utt;
        q = 0;
        upairs = pairs_in(p, utt);
      }
      fetch();
    }
    // checked build: the Mel rounds read inside the padded power array and write inside the
    // utterance's rows of the result
    if (!PREBA_IN_RANGE(p.status,
                        mel_begin[0] >= 0 && mel_begin[0] + static_cast<int>(kMelIters0) <= static_cast<int>(kPowLen) &&
                            mel_begin[1] >= 0 && mel_begin[1] + static_cast<int>(kMelIters1) <= static_cast<int>(kPowLen) &&
                            mel_begin[2] >= 0 && mel_begin[2] + static_cast<int>(kMelIters2) <= static_cast<int>(kPowLen) &&
                            (mel_filter[0] == 0xffu || mel_filter[0] < kMels) &&
                            (mel_filter[1] == 0xffu || mel_filter[1] < kMels) &&
                            (mel_filter[2] == 0xffu || mel_filter[2] < kMels) &&
                            this_t0 + (have1 ? 1u : 0u) < p.t_max)) {
      __syncwarp();
      continue;
    }
    mel_round<kMelIters0>(plan.w + lane, ws.power + mel_begin[0], mel_filter[0], out, p.t_max,
                          this_t0, have1);
    mel_round<kMelIters1>(plan.w + kMelIters0 * 32 + lane, ws.power + mel_begin[1], mel_filter[1],
                          out, p.t_max, this_t0, have1);
    mel_round<kMelIters2>(plan.w + (kMelIters0 + kMelIters1) * 32 + lane, ws.power + mel_begin[2],
                          mel_filter[2], out, p.t_max, this_t0, have1);
    __syncwarp();  // the next pair reuses this warp's buffers
  }

  // zeros behind every utterance's own frames: rows dealt out to the warps in turn
  const uint64_t rows = static_cast<uint64_t>(p.n) * kMels;
  for (uint64_t row = gwarp; row < rows; row += nwarps) {
    const uint32_t i = static_cast<uint32_t>(row / kMels);
    const uint32_t frames = frames_in(p, i);
    float* __restrict__ o = p.out + row * p.t_max;
    for (uint32_t t = frames + lane; t < p.t_max; t += 32) o[t] = 0.f;
  }
  // A launch marked as overlapping started without waiting for the kernels before it on the
  // stream; it does not complete before them (stream order of completion is kept).
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (gwarp == 0) {  // refused entries are reported once
    bool bad = false;
    for (uint32_t i = lane; i < p.n; i += 32) bad |= !utt_ok(p.table[i], p.samples_count);
    if (__any_sync(0xffffffffu, bad) && lane == 0 && p.status)
      atomicCAS(p.status, 0, PREBA_ERR_BAD_TABLE);
  }
}

// Normalize: a warp per (utterance, filter) row; rows of up to 32 * kHold frames stay in
// registers between the three passes.
constexpr int kHold = 48;

__global__ void __launch_bounds__(256) normalize_kernel(const AudioParams p) {
  // launched as a programmatic dependent of the spectrogram kernel: let the launch behind
  // this one be scheduled (a spectrogram marked as overlapping moves in as these CTAs retire),
  // then wait for the spectrogram's results
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const uint32_t lane = threadIdx.x & 31;
  const uint32_t row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (row >= p.n * kMels) return;
  const uint32_t utt = row / kMels;
  const uint32_t frames = frames_in(p, utt);
  if (frames == 0) return;
  float* __restrict__ r = p.out + static_cast<size_t>(row) * p.t_max;
  const float count = static_cast<float>(frames);
  if (frames <= 32u * kHold) {
    float hold[kHold];
    float sum = 0.f;
#pragma unroll
    for (int i = 0; i < kHold; ++i) {
      const uint32_t t = lane + 32u * i;
      hold[i] = t < frames ? r[t] : 0.f;
      sum += hold[i];
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    const float mean = sum / count;
    float sq = 0.f;
#pragma unroll
    for (int i = 0; i < kHold; ++i) {
      const float d = lane + 32u * i < frames ? hold[i] - mean : 0.f;
      hold[i] = d;
      sq = fmaf(d, d, sq);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
    const float inv = 1.0f / (sqrtf(sq / count) + kStdGuard);
#pragma unroll
    for (int i = 0; i < kHold; ++i) {
      const uint32_t t = lane + 32u * i;
      if (t < frames) r[t] = hold[i] * inv;
    }
    return;
  }
  float sum = 0.f;
  for (uint32_t t = lane; t < frames; t += 32) sum += r[t];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
  const float mean = sum / count;
  float sq = 0.f;
  for (uint32_t t = lane; t < frames; t += 32) {
    const float d = r[t] - mean;
    sq = fmaf(d, d, sq);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
  const float inv = 1.0f / (sqrtf(sq / count) + kStdGuard);
  for (uint32_t t = lane; t < frames; t += 32) r[t] = (r[t] - mean) * inv;
}

}  // namespace audio
}  // namespace preba

extern "C" int preba_audio_query(const uint32_t* lengths, uint32_t n, preba_audio_sizes_t* sizes) {
  if (!lengths || !sizes || n == 0) return PREBA_ERR_INVALID_ARG;
  uint64_t at = 0;
  uint32_t t_max = 0;
  for (uint32_t i = 0; i < n; ++i) {
    if (lengths[i] > PREBA_AUDIO_MAX_SAMPLES) return PREBA_ERR_INVALID_ARG;
    at = preba::align_up(at + lengths[i], PREBA_AUDIO_ALIGN);
    const uint32_t f = preba::audio::frames_of(lengths[i]);
    t_max = f > t_max ? f : t_max;
  }
  sizes->packed_samples = at;
  sizes->table_bytes = static_cast<uint64_t>(n) * sizeof(preba_utt_t);
  sizes->out_bytes = static_cast<uint64_t>(n) * PREBA_AUDIO_MELS * t_max * sizeof(float);
  sizes->t_max = t_max;
  sizes->reserved = 0;
  return PREBA_OK;
}

extern "C" int preba_audio_pack(const float* const* utterances, const uint32_t* lengths,
                                uint32_t n, float* packed, uint64_t capacity_samples,
                                preba_utt_t* table) {
  if (!utterances || !lengths || !packed || !table || n == 0) return PREBA_ERR_INVALID_ARG;
  uint64_t need = 0;
  for (uint32_t i = 0; i < n; ++i) {
    if ((!utterances[i] && lengths[i]) || lengths[i] > PREBA_AUDIO_MAX_SAMPLES)
      return PREBA_ERR_INVALID_ARG;
    need = preba::align_up(need + lengths[i], PREBA_AUDIO_ALIGN);
  }
  if (capacity_samples < need) return PREBA_ERR_BUFFER_TOO_SMALL;
  uint64_t at = 0;
  for (uint32_t i = 0; i < n; ++i) {
    table[i].offset = at;
    table[i].length = lengths[i];
    table[i].frames = preba::audio::frames_of(lengths[i]);
    if (lengths[i]) std::memcpy(packed + at, utterances[i], sizeof(float) * lengths[i]);
    const uint64_t next = preba::align_up(at + lengths[i], PREBA_AUDIO_ALIGN);
    for (uint64_t k = at + lengths[i]; k < next; ++k) packed[k] = 0.0f;
    at = next;
  }
  return PREBA_OK;
}

namespace preba {
namespace audio {

// ---- Resample: bandlimited interpolation with a Hann-windowed sinc ---------------------------------
constexpr uint32_t kResampleZeros = 6;
constexpr float kResampleRolloff = 0.99f;
constexpr uint32_t kResampleChunk = 2048;        // output samples per CTA
constexpr uint32_t kResampleTableMax = 12000;    // floats of shared memory for the phase table

struct ResampleParams {
  const float* in;
  uint64_t in_count;
  const preba_utt_t* table_in;
  float* out;
  uint64_t out_count;
  const preba_utt_t* table_out;
  int32_t* status;
  uint32_t n;
  uint32_t orig, fresh;  // the two rates divided by their greatest common divisor
  uint32_t reach;        // taps reach from centre - reach to centre + reach + 1
  float fc;              // cutoff relative to the input rate
};

// Output sample m of an utterance sits at position m * orig / fresh of the input; with
// centre = floor of that and phase p = (m * orig) mod fresh, its value is
// sum_j x[centre - reach + j] * h((j - reach) - p / fresh).  A CTA tabulates h for every
// phase once and then produces a run of outputs.
__global__ void __launch_bounds__(256) resample_kernel(const ResampleParams p) {
  __shared__ float table[kResampleTableMax];
  const uint32_t taps = 2 * p.reach + 2;
  const preba_utt_t ui = p.table_in[blockIdx.y], uo = p.table_out[blockIdx.y];
  const uint64_t want = (static_cast<uint64_t>(ui.length) * p.fresh + p.orig - 1) / p.orig;
  const bool ok = ui.offset % PREBA_AUDIO_ALIGN == 0 && uo.offset % PREBA_AUDIO_ALIGN == 0 &&
                  ui.offset <= p.in_count && ui.length <= p.in_count - ui.offset &&
                  uo.length == want && uo.offset <= p.out_count &&
                  (static_cast<uint64_t>(uo.length) + 3) / 4 * 4 <= p.out_count - uo.offset;
  if (!ok) {
    if (threadIdx.x == 0 && blockIdx.x == 0 && p.status)
      atomicCAS(p.status, 0, PREBA_ERR_BAD_TABLE);
    return;
  }
  const uint32_t m0 = blockIdx.x * kResampleChunk;
  const uint32_t padded = (uo.length + 3) / 4 * 4;  // alignment padding is written as 0
  if (m0 >= padded) return;
  for (uint32_t i = threadIdx.x; i < p.fresh * taps; i += blockDim.x) {
    const uint32_t phase = i / taps, j = i - phase * taps;
    const float t = (static_cast<float>(j) - static_cast<float>(p.reach)) -
                    static_cast<float>(phase) / static_cast<float>(p.fresh);
    const float u = p.fc * t;
    float h = 0.f;
    if (fabsf(u) < static_cast<float>(kResampleZeros)) {
      const float sinc = u == 0.f ? 1.0f : sinpif(u) / (3.14159265358979323846f * u);
      const float c = cospif(u / (2.0f * kResampleZeros));
      h = p.fc * sinc * c * c;
    }
    table[i] = h;
  }
  __syncthreads();
  const float* __restrict__ x = p.in + ui.offset;
  float* __restrict__ y = p.out + uo.offset;
  const uint32_t m_end = min(m0 + kResampleChunk, padded);
  for (uint32_t m = m0 + threadIdx.x; m < m_end; m += blockDim.x) {
    float acc = 0.f;
    if (m < uo.length) {
      const uint64_t pos = static_cast<uint64_t>(m) * p.orig;
      const uint32_t centre = static_cast<uint32_t>(pos / p.fresh);
      const float* __restrict__ h = table + (pos - static_cast<uint64_t>(centre) * p.fresh) * taps;
      if (centre >= p.reach && centre - p.reach + taps <= ui.length) {
        // every tap lies inside the utterance
        const float* __restrict__ xs = x + (centre - p.reach);
#pragma unroll 4
        for (uint32_t j = 0; j < taps; ++j) acc = fmaf(xs[j], h[j], acc);
      } else {
        const int64_t first = static_cast<int64_t>(centre) - p.reach;
        for (uint32_t j = 0; j < taps; ++j) {
          const int64_t idx = first + j;
          if (idx >= 0 && idx < static_cast<int64_t>(ui.length)) acc = fmaf(x[idx], h[j], acc);
        }
      }
    }
    y[m] = acc;
  }
}

uint32_t gcd32(uint32_t a, uint32_t b) {
  while (b) {
    const uint32_t r = a % b;
    a = b;
    b = r;
  }
  return a;
}

}  // namespace audio
}  // namespace preba

extern "C" int preba_audio_layout(const uint32_t* lengths, uint32_t n, preba_utt_t* table) {
  if (!lengths || !table || n == 0) return PREBA_ERR_INVALID_ARG;
  uint64_t at = 0;
  for (uint32_t i = 0; i < n; ++i) {
    if (lengths[i] > PREBA_AUDIO_MAX_SAMPLES) return PREBA_ERR_INVALID_ARG;
    table[i].offset = at;
    table[i].length = lengths[i];
    table[i].frames = preba::audio::frames_of(lengths[i]);
    at = preba::align_up(at + lengths[i], PREBA_AUDIO_ALIGN);
  }
  return PREBA_OK;
}

extern "C" int preba_audio_resample_query(const uint32_t* lengths_in, uint32_t n, uint32_t rate_in,
                                          uint32_t rate_out, uint32_t* lengths_out) {
  if (!lengths_in || !lengths_out || n == 0 || rate_in == 0 || rate_out == 0)
    return PREBA_ERR_INVALID_ARG;
  const uint32_t g = preba::audio::gcd32(rate_in, rate_out);
  const uint64_t orig = rate_in / g, fresh = rate_out / g;
  for (uint32_t i = 0; i < n; ++i) {
    const uint64_t m = (lengths_in[i] * fresh + orig - 1) / orig;
    if (lengths_in[i] > PREBA_AUDIO_MAX_SAMPLES || m > PREBA_AUDIO_MAX_SAMPLES)
      return PREBA_ERR_INVALID_ARG;
    lengths_out[i] = static_cast<uint32_t>(m);
  }
  return PREBA_OK;
}

extern "C" int preba_audio_resample(const float* samples_in, uint64_t samples_in_count,
                                    const preba_utt_t* table_in, float* samples_out,
                                    uint64_t samples_out_count, const preba_utt_t* table_out,
                                    uint32_t n, uint32_t longest_out, uint32_t rate_in,
                                    uint32_t rate_out, int32_t* status, void* stream) {
  using namespace preba::audio;
  if (!samples_in || !table_in || !samples_out || !table_out || n == 0 || n > 65535 ||
      rate_in == 0 || rate_out == 0 || longest_out > PREBA_AUDIO_MAX_SAMPLES)
    return PREBA_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(samples_in) % 16 || reinterpret_cast<uintptr_t>(samples_out) % 16)
    return PREBA_ERR_INVALID_ARG;
  ResampleParams p;
  const uint32_t g = gcd32(rate_in, rate_out);
  p.orig = rate_in / g;
  p.fresh = rate_out / g;
  const double fc = static_cast<double>(kResampleRolloff) *
                    (p.fresh < p.orig ? static_cast<double>(p.fresh) / p.orig : 1.0);
  p.fc = static_cast<float>(fc);
  p.reach = static_cast<uint32_t>(std::ceil(kResampleZeros / fc)) + 1;
  if (static_cast<uint64_t>(p.fresh) * (2 * p.reach + 2) > kResampleTableMax)
    return PREBA_ERR_INVALID_ARG;  // the phase table of this rate pair does not fit
  p.in = samples_in;
  p.in_count = samples_in_count;
  p.table_in = table_in;
  p.out = samples_out;
  p.out_count = samples_out_count;
  p.table_out = table_out;
  p.status = status;
  p.n = n;
  if (longest_out == 0) return PREBA_OK;
  const dim3 grid((longest_out + 3 + kResampleChunk - 1) / kResampleChunk, n);
  resample_kernel<<<grid, 256, 0, static_cast<cudaStream_t>(stream)>>>(p);
  const cudaError_t err = cudaGetLastError();
  if (err != cudaSuccess) {
    preba::g_last_cuda_error = static_cast<int>(err);
    return PREBA_ERR_CUDA;
  }
  return PREBA_OK;
}

namespace preba {
namespace audio {

// CTAs of the spectrogram kernel the current device holds at once (the grid of its persistent
// launch); computed once per device and kept (concurrent first calls store the same value).
int resident_ctas(cudaError_t* err) {
  constexpr int kMaxDevices = 64;
  static std::atomic<int> cache[kMaxDevices];
  int dev = 0;
  *err = cudaGetDevice(&dev);
  if (*err != cudaSuccess) return 0;
  if (dev >= 0 && dev < kMaxDevices) {
    const int known = cache[dev].load(std::memory_order_relaxed);
    if (known > 0) return known;
  }
  int sms = 0, per_sm = 0;
  *err = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (*err != cudaSuccess) return 0;
  *err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, logmel_kernel, 32 * kWarps, 0);
  if (*err != cudaSuccess) return 0;
  const int resident = sms * (per_sm > 0 ? per_sm : 1);
  if (dev >= 0 && dev < kMaxDevices) cache[dev].store(resident, std::memory_order_relaxed);
  return resident;
}

}  // namespace audio
}  // namespace preba

extern "C" int preba_audio_logmel(const preba_audio_batch_t* b, int normalize, void* stream) {
  using namespace preba::audio;
  if (!b || !b->samples || !b->table || !b->out || b->n == 0 || b->n > 65535 || b->t_max == 0 ||
      (normalize & ~(PREBA_AUDIO_NORMALIZE | PREBA_AUDIO_OVERLAP_PREVIOUS)) != 0)
    return PREBA_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(b->samples) % 16 || reinterpret_cast<uintptr_t>(b->out) % 4 ||
      reinterpret_cast<uintptr_t>(b->table) % 8)
    return PREBA_ERR_INVALID_ARG;
  const uint64_t need = static_cast<uint64_t>(b->n) * kMels * b->t_max * sizeof(float);
  if (b->out_bytes < need) return PREBA_ERR_BUFFER_TOO_SMALL;
  if (static_cast<uint64_t>(b->n) * kMels * b->t_max > 0xffffffffull) return PREBA_ERR_INVALID_ARG;
  if (b->table_host) {
    for (uint32_t i = 0; i < b->n; ++i) {
      const preba_utt_t& u = b->table_host[i];
      if (u.offset % PREBA_AUDIO_ALIGN || u.length > PREBA_AUDIO_MAX_SAMPLES ||
          u.offset > b->samples_count || u.length > b->samples_count - u.offset ||
          u.frames != frames_of(u.length) || u.frames > b->t_max)
        return PREBA_ERR_BAD_TABLE;
    }
  }
  static const MelPlan mel = make_mel_plan();
  if (!mel.ok) return PREBA_ERR_INVALID_ARG;  // cannot happen for the constants above
  AudioParams p;
  p.samples = b->samples;
  p.samples_count = b->samples_count;
  p.table = b->table;
  p.out = b->out;
  p.status = b->status;
  p.n = b->n;
  p.t_max = b->t_max;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // persistent grid: what the device holds at once, but no more warps than a few frame pairs
  // each would keep busy (an upper bound on the pairs: half of t_max, rounded up, per entry)
  cudaError_t err = cudaSuccess;
  const int resident = resident_ctas(&err);
  if (err == cudaSuccess) {
    const uint64_t pairs = static_cast<uint64_t>(b->n) * ((b->t_max + 1) / 2);
    const uint64_t want = (pairs + 2 * kWarps - 1) / (2 * kWarps);
    const uint32_t blocks = static_cast<uint32_t>(
        std::max<uint64_t>(1, std::min<uint64_t>(want, static_cast<uint64_t>(resident))));
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(blocks);
    cfg.blockDim = dim3(32 * kWarps);
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = (normalize & PREBA_AUDIO_OVERLAP_PREVIOUS) ? 1 : 0;
    err = cudaLaunchKernelEx(&cfg, logmel_kernel, p, mel);
  }
  if (err == cudaSuccess && (normalize & PREBA_AUDIO_NORMALIZE)) {
    const uint32_t rows = b->n * kMels;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((rows + 7) / 8);
    cfg.blockDim = dim3(256);
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    err = cudaLaunchKernelEx(&cfg, normalize_kernel, p);
  }
  if (err != cudaSuccess) {
    preba::g_last_cuda_error = static_cast<int>(err);
    return PREBA_ERR_CUDA;
  }
  return PREBA_OK;
}
