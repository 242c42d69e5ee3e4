// Audio path: log Mel spectrogram and per-utterance normalisation of a ragged batch (sm_100a).
//
// Kernel 1: a warp takes two consecutive frames of one utterance, multiplies them by the Hann
// window, packs them as the real and imaginary part of one complex sequence, runs a 512-point
// FFT as three passes of radix-8 butterflies in registers (exchanging through its own shared
// memory between passes), separates the two spectra, forms the power spectra,
// applies the triangular Mel filters (a lane per filter, the filter's few bins read from
// shared memory) and writes log(energy + 2^-24).  Frames past an utterance's own count are
// written as 0, so the result tensor needs no clearing.
// Kernel 2 (Normalize): a warp per (utterance, filter) row makes the paper's three passes:
// mean, variance from that mean, normalisation.
// fp32 throughout; the path is bound by arithmetic and shared memory, not by HBM.
#include <cuda_runtime.h>

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
constexpr int kPairsPerWarp = 4;      // frame pairs a warp transforms one after the other
constexpr int kFramesPerCta = 2 * kWarps * kPairsPerWarp;
constexpr float kLogGuard = 5.9604644775390625e-08f;  // 2^-24
constexpr float kStdGuard = 1e-5f;

// The Mel filters in the form the kernel uses: filter j covers the consecutive bins
// first[j] .. first[j] + count[j] - 1 and their weights lie one after the other in w from
// start[j] (rising edge, then falling edge; every bin belongs to at most two filters).
constexpr uint32_t kMelWeights = 2 * kBins + 2;
struct MelTable {
  float w[kMelWeights];
  uint16_t first[kMels];
  uint16_t count[kMels];
  uint16_t start[kMels];
};
static_assert(sizeof(MelTable) % 4 == 0 && sizeof(MelTable) < 3800, "passed as a kernel parameter");

uint32_t frames_of(uint32_t length) { return length < kWin ? 0u : 1u + (length - kWin) / kHop; }

// Corner frequencies equally spaced on the HTK mel scale between 0 and rate / 2 (double);
// filter j rises from corner j to corner j + 1 and falls to corner j + 2.
MelTable make_mel_table() {
  MelTable t;
  std::memset(&t, 0, sizeof(t));
  const double top = 2595.0 * std::log10(1.0 + (PREBA_AUDIO_RATE / 2.0) / 700.0);
  double corner[kMels + 2];
  for (uint32_t i = 0; i < kMels + 2; ++i)
    corner[i] = 700.0 * (std::pow(10.0, (top * i / (kMels + 1)) / 2595.0) - 1.0);
  corner[0] = 0.0;
  corner[kMels + 1] = PREBA_AUDIO_RATE / 2.0;
  uint32_t at = 0;
  for (uint32_t j = 0; j < kMels; ++j) {
    const double lo = corner[j], mid = corner[j + 1], hi = corner[j + 2];
    t.start[j] = static_cast<uint16_t>(at);
    bool any = false;
    for (uint32_t k = 0; k < kBins; ++k) {
      const double f = static_cast<double>(k) * PREBA_AUDIO_RATE / kFft;
      if (f <= lo || f >= hi) continue;  // weight 0 at and beyond the feet
      const double wgt = f < mid ? (f - lo) / (mid - lo) : (hi - f) / (hi - mid);
      if (!any) t.first[j] = static_cast<uint16_t>(k);
      any = true;
      if (at < kMelWeights) t.w[at++] = static_cast<float>(wgt);
      t.count[j] = static_cast<uint16_t>(k + 1 - t.first[j]);
    }
  }
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

// The 512-point FFT runs as three passes of radix-8 butterflies held in registers
// (512 = 8 * 8 * 8); between passes the warp exchanges its values through an 8 x 64 array in
// shared memory whose rows are 68 elements apart, which keeps every exchange at the two
// wavefronts a 64-bit access of 32 lanes needs.
constexpr uint32_t kPitch = 68;

struct __align__(16) WarpFft {
  float2 z[8 * kPitch];  // exchange array, then the spectrum in natural order (first 512)
  float2 power[kBins + 1];  // the two frames' power spectra side by side
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

__global__ void __launch_bounds__(32 * kWarps)
logmel_kernel(const AudioParams p, const MelTable mel_param) {
  __shared__ WarpFft sm[kWarps];
  __shared__ float2 twiddle[kFft];  // exp(-2 pi i j / 512)
  __shared__ float window[kWin];
  __shared__ MelTable mel;  // lanes read different entries: shared memory, not the constant bank
  const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const uint32_t utt = blockIdx.y;
  const preba_utt_t u = p.table[utt];
  const bool ok = utt_ok(u, p.samples_count);
  if (!ok && threadIdx.x == 0 && blockIdx.x == 0 && p.status)
    atomicCAS(p.status, 0, PREBA_ERR_BAD_TABLE);
  const uint32_t frames = ok ? min(u.frames, p.t_max) : 0u;
  float* __restrict__ out = p.out + static_cast<size_t>(utt) * kMels * p.t_max;
  const uint32_t cta_t0 = blockIdx.x * kFramesPerCta;
  if (cta_t0 >= frames) {
    // padding (or a refused entry): zeros for all of this CTA's frames
    const uint32_t t_end = min(cta_t0 + kFramesPerCta, p.t_max);
    for (uint32_t j = warp; j < kMels; j += kWarps)
      for (uint32_t t = cta_t0 + lane; t < t_end; t += 32) out[static_cast<size_t>(j) * p.t_max + t] = 0.f;
    return;
  }
  for (uint32_t k = threadIdx.x; k < kFft; k += blockDim.x) {
    float s, c;
    sincospif(-2.0f * static_cast<float>(k) / kFft, &s, &c);
    twiddle[k] = make_float2(c, s);
  }
  for (uint32_t i = threadIdx.x; i < kWin; i += blockDim.x)
    window[i] = 0.5f - 0.5f * cospif(2.0f * static_cast<float>(i) / kWin);
  {
    const uint32_t* src = reinterpret_cast<const uint32_t*>(&mel_param);
    uint32_t* dst = reinterpret_cast<uint32_t*>(&mel);
    for (uint32_t i = threadIdx.x; i < sizeof(MelTable) / 4; i += blockDim.x) dst[i] = src[i];
  }
  __syncthreads();

  WarpFft& ws = sm[warp];
#pragma unroll 1
  for (uint32_t pair = 0; pair < kPairsPerWarp; ++pair) {
    const uint32_t t0 = cta_t0 + 2 * (warp + kWarps * pair);  // this warp's two frames
    if (t0 >= p.t_max) break;
    const bool have0 = t0 < frames, have1 = t0 + 1 < frames;
    if (!have0) {
      for (uint32_t j = lane; j < kMels; j += 32) {
        out[static_cast<size_t>(j) * p.t_max + t0] = 0.f;
        if (t0 + 1 < p.t_max) out[static_cast<size_t>(j) * p.t_max + t0 + 1] = 0.f;
      }
      continue;
    }
    const float* __restrict__ x = p.samples + u.offset + static_cast<size_t>(t0) * kHop;
    // With n = 64 n2 + 8 n1 + n0 and k = k0 + 8 k1 + 64 k2:
    //   X[k] = sum_n0 W8^(n0 k2) W512^(n0 (k0 + 8 k1))
    //          sum_n1 W8^(n1 k1) W64^(n1 k0) sum_n2 W8^(n2 k0) x[n].
    // Pass 1 (over n2): a lane takes the columns p = 8 n1 + n0 = lane and lane + 32 of the two
    // windowed frames (real and imaginary part).
    float2 v[2][8];
#pragma unroll
    for (int c = 0; c < 2; ++c) {
      const uint32_t pcol = lane + 32 * c;
#pragma unroll
      for (uint32_t n2 = 0; n2 < 8; ++n2) {
        const uint32_t i = 64 * n2 + pcol;
        float re = 0.f, im = 0.f;
        if (i < kWin) {
          re = x[i] * window[i];
          if (have1) im = x[i + kHop] * window[i];
        }
        v[c][n2] = make_float2(re, im);
      }
      fft8(v[c]);
      const uint32_t n1 = pcol >> 3;
#pragma unroll
      for (uint32_t k0 = 0; k0 < 8; ++k0)
        ws.z[k0 * kPitch + pcol] = k0 ? cmul(v[c][k0], twiddle[8 * n1 * k0]) : v[c][0];
    }
    __syncwarp();
    // Pass 2 (over n1): a lane takes q = 8 k0 + n0.
#pragma unroll
    for (int c = 0; c < 2; ++c) {
      const uint32_t q = lane + 32 * c, k0 = q >> 3, n0 = q & 7;
#pragma unroll
      for (uint32_t n1 = 0; n1 < 8; ++n1) v[c][n1] = ws.z[k0 * kPitch + 8 * n1 + n0];
    }
    __syncwarp();
#pragma unroll
    for (int c = 0; c < 2; ++c) {
      const uint32_t q = lane + 32 * c, k0 = q >> 3, n0 = q & 7;
      fft8(v[c]);
#pragma unroll
      for (uint32_t k1 = 0; k1 < 8; ++k1)
        ws.z[n0 * kPitch + k0 + 8 * k1] = cmul(v[c][k1], twiddle[n0 * (k0 + 8 * k1)]);
    }
    __syncwarp();
    // Pass 3 (over n0): a lane takes r = k0 + 8 k1 and produces X[r + 64 k2].
#pragma unroll
    for (int c = 0; c < 2; ++c) {
      const uint32_t r = lane + 32 * c;
#pragma unroll
      for (uint32_t n0 = 0; n0 < 8; ++n0) v[c][n0] = ws.z[n0 * kPitch + r];
    }
    __syncwarp();
#pragma unroll
    for (int c = 0; c < 2; ++c) {
      const uint32_t r = lane + 32 * c;
      fft8(v[c]);
#pragma unroll
      for (uint32_t k2 = 0; k2 < 8; ++k2) ws.z[r + 64 * k2] = v[c][k2];
    }
    __syncwarp();
    // Z = A + iB with A, B the spectra of the two real frames:
    // A[k] = (Z[k] + conj(Z[N-k]))/2, B[k] = (Z[k] - conj(Z[N-k]))/(2i)
    for (uint32_t k = lane; k < kBins; k += 32) {
      const float2 zk = ws.z[k], zn = ws.z[(kFft - k) & (kFft - 1)];
      const float ar = 0.5f * (zk.x + zn.x), ai = 0.5f * (zk.y - zn.y);
      const float br = 0.5f * (zk.y + zn.y), bi = 0.5f * (zn.x - zk.x);
      ws.power[k] = make_float2(ar * ar + ai * ai, br * br + bi * bi);
    }
    __syncwarp();
    for (uint32_t j = lane; j < kMels; j += 32) {
      float e0 = 0.f, e1 = 0.f;
      const uint32_t first = mel.first[j], count = mel.count[j], start = mel.start[j];
      for (uint32_t i = 0; i < count; ++i) {
        const float wgt = mel.w[start + i];
        const float2 pw = ws.power[first + i];
        e0 = fmaf(wgt, pw.x, e0);
        e1 = fmaf(wgt, pw.y, e1);
      }
      out[static_cast<size_t>(j) * p.t_max + t0] = logf(e0 + kLogGuard);
      if (t0 + 1 < p.t_max)
        out[static_cast<size_t>(j) * p.t_max + t0 + 1] = have1 ? logf(e1 + kLogGuard) : 0.f;
    }
    __syncwarp();  // the next pair reuses this warp's buffers
  }
}

// Normalize: a warp per (utterance, filter) row.
__global__ void __launch_bounds__(128) normalize_kernel(const AudioParams p) {
  const uint32_t lane = threadIdx.x & 31;
  const uint32_t row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (row >= p.n * kMels) return;
  const uint32_t utt = row / kMels;
  const preba_utt_t u = p.table[utt];
  if (!utt_ok(u, p.samples_count)) return;
  const uint32_t frames = min(u.frames, p.t_max);
  if (frames == 0) return;
  float* __restrict__ r = p.out + static_cast<size_t>(row) * p.t_max;
  float sum = 0.f;
  for (uint32_t t = lane; t < frames; t += 32) sum += r[t];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
  const float mean = sum / static_cast<float>(frames);
  float sq = 0.f;
  for (uint32_t t = lane; t < frames; t += 32) {
    const float d = r[t] - mean;
    sq = fmaf(d, d, sq);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
  const float inv = 1.0f / (sqrtf(sq / static_cast<float>(frames)) + kStdGuard);
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

extern "C" int preba_audio_logmel(const preba_audio_batch_t* b, int normalize, void* stream) {
  using namespace preba::audio;
  if (!b || !b->samples || !b->table || !b->out || b->n == 0 || b->n > 65535 || b->t_max == 0)
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
  static const MelTable mel = make_mel_table();
  AudioParams p;
  p.samples = b->samples;
  p.samples_count = b->samples_count;
  p.table = b->table;
  p.out = b->out;
  p.status = b->status;
  p.n = b->n;
  p.t_max = b->t_max;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const dim3 grid((b->t_max + kFramesPerCta - 1) / kFramesPerCta, b->n);
  logmel_kernel<<<grid, 32 * kWarps, 0, s>>>(p, mel);
  cudaError_t err = cudaGetLastError();
  if (err == cudaSuccess && normalize) {
    const uint32_t rows = b->n * kMels;
    normalize_kernel<<<(rows + 3) / 4, 128, 0, s>>>(p);
    err = cudaGetLastError();
  }
  if (err != cudaSuccess) {
    preba::g_last_cuda_error = static_cast<int>(err);
    return PREBA_ERR_CUDA;
  }
  return PREBA_OK;
}
