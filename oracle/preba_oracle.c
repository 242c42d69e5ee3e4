/*
 * TEST INFRASTRUCTURE ONLY — the CPU oracle for the vision preprocessing path
 * (resize -> center crop -> normalise -> HWC->NCHW).
 *
 * This file is the plain, slow, double-precision statement of what the path
 * computes.  It is used by the tests, by the smoke check and by the benchmark's
 * CPU-baseline leg, and by nothing else: the product library never links it,
 * and it shares no code, header or table with the CUDA path.
 *
 * What it follows.  The paper (Sec. 2.3 item 1; Fig. 4; Table 1 rows "Resize",
 * "Crop", "Normalize") names the operations and their order: a decoded RGB
 * image is resized, cropped to the model's input size (e.g. 224x224x3) and
 * normalised; Sec. 4.2 states that each operation consumes only the previous
 * one's output, and that requests are independent single inputs.  The paper
 * does not state the interpolation kernel, the rounding of the resized size,
 * the crop origin or the normalisation constants; the readings taken here are
 *   - shorter side -> S, longer side -> floor(S*long/short);
 *   - bilinear, half-pixel centres, edge clamp, no antialias, per-axis
 *     in/out ratio as the sampling scale;
 *   - crop origin floor((R-C)/2) on both axes;
 *   - no intermediate rounding: out = (v/255 - mean_c)/std_c on the real v;
 *   - channel c of the input goes to plane c of the output.
 * Because none of this is an approximation, the oracle is the definition
 * written out, element by element, with exact integer sampling geometry and
 * double arithmetic.
 *
 * Every function here is pinned by tests that do not call it to make their
 * expected values (identity, pure crop, constant images, ramp upscales, affine
 * reproduction, exact-rational brute force, hand-worked pixels, a library
 * special case): no function is "parity unpinned".
 */
#include <math.h>
#include <pthread.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_OK 0
#define ORACLE_ERR_ARG -1
#define ORACLE_ERR_SPACE -2

#define ORACLE_PACK_ALIGN 128u /* start of every image, and the total, are multiples of this */

/* Resized size of an (h, w) image whose shorter side becomes s:
 * the longer side is floor(s * long / short).  (Resize unit, Table 1.) */
int oracle_resized_size(uint32_t h, uint32_t w, uint32_t s, uint64_t* rh, uint64_t* rw) {
  if (h == 0 || w == 0 || s == 0 || !rh || !rw) return ORACLE_ERR_ARG;
  if (h <= w) {
    *rh = s;
    *rw = ((uint64_t)s * w) / h;
  } else {
    *rw = s;
    *rh = ((uint64_t)s * h) / w;
  }
  return ORACLE_OK;
}

/* One axis of the sampling grid.  Output index j of the crop window (size c)
 * sits at index X = j + floor((r - c)/2) of the resized axis (length r); its
 * centre maps to source coordinate sx = (X + 1/2) * in / r - 1/2, clamped to
 * [0, in-1].  In exact integers: sx = num/den with num = (2X+1)*in - r,
 * den = 2r.  Returns the two taps and the weight of the second one. */
int oracle_axis(uint32_t in, uint64_t r, uint32_t c, uint32_t j,
                uint32_t* i0, uint32_t* i1, double* lambda) {
  if (in == 0 || r < c || j >= c || !i0 || !i1 || !lambda) return ORACLE_ERR_ARG;
  const uint64_t origin = (r - c) / 2;
  const uint64_t X = origin + j;
  const int64_t den = 2 * (int64_t)r;
  int64_t num = (2 * (int64_t)X + 1) * (int64_t)in - (int64_t)r;
  const int64_t hi = ((int64_t)in - 1) * den;
  if (num < 0) num = 0;
  if (num > hi) num = hi;
  const int64_t q = num / den;
  const int64_t rem = num % den;
  *i0 = (uint32_t)q;
  *i1 = (uint32_t)((q + 1 < (int64_t)in) ? q + 1 : (int64_t)in - 1);
  *lambda = (double)rem / (double)den;
  return ORACLE_OK;
}

/* One output element out[ch][k][j] of one image (HWC uint8, row pitch 3*w).
 * Bilinear value in difference form, so that equal taps give the tap exactly;
 * then the normalisation, with mean/std widened from the caller's floats. */
int oracle_element(const uint8_t* img, uint32_t h, uint32_t w, uint32_t c, uint32_t s,
                   const float mean[3], const float std[3],
                   uint32_t ch, uint32_t k, uint32_t j, double* out) {
  uint64_t rh, rw;
  if (!img || !out || !mean || !std || ch > 2) return ORACLE_ERR_ARG;
  if (oracle_resized_size(h, w, s, &rh, &rw) != ORACLE_OK) return ORACLE_ERR_ARG;
  uint32_t x0, x1, y0, y1;
  double lx, ly;
  if (oracle_axis(w, rw, c, j, &x0, &x1, &lx) != ORACLE_OK) return ORACLE_ERR_ARG;
  if (oracle_axis(h, rh, c, k, &y0, &y1, &ly) != ORACLE_OK) return ORACLE_ERR_ARG;
  const size_t pitch = (size_t)3 * w;
  const double p00 = img[y0 * pitch + 3 * (size_t)x0 + ch];
  const double p01 = img[y0 * pitch + 3 * (size_t)x1 + ch];
  const double p10 = img[y1 * pitch + 3 * (size_t)x0 + ch];
  const double p11 = img[y1 * pitch + 3 * (size_t)x1 + ch];
  const double a = p00 + lx * (p01 - p00);
  const double b = p10 + lx * (p11 - p10);
  const double v = a + ly * (b - a);
  *out = (v / 255.0 - (double)mean[ch]) / (double)std[ch];
  return ORACLE_OK;
}

/* Round a double once to IEEE binary16, ties to even; returns the bit pattern.
 * Written from the format: 1 sign, 5 exponent (bias 15), 10 fraction bits;
 * subnormals are multiples of 2^-24; values that round to >= 65520 overflow
 * to infinity. */
uint16_t oracle_round_f16(double x) {
  const uint16_t sign = signbit(x) ? 0x8000u : 0u;
  if (isnan(x)) return (uint16_t)(sign | 0x7e00u);
  double a = fabs(x);
  if (isinf(a)) return (uint16_t)(sign | 0x7c00u);
  if (a == 0.0) return sign;
  int e;
  (void)frexp(a, &e); /* a = m * 2^e, m in [0.5, 1)  => a in [2^(e-1), 2^e) */
  int exp2 = e - 1;   /* unbiased exponent of the leading bit */
  if (exp2 < -14) exp2 = -14; /* subnormal range shares the spacing 2^-24 */
  /* spacing of representable values around a: 2^(exp2-10) */
  const double q = ldexp(a, 10 - exp2); /* a in units of the spacing; exact */
  double n = nearbyint(q);              /* default mode: ties to even */
  /* units -> bits: a normal value with exponent exp2 has n in [1024, 2048] */
  uint64_t units = (uint64_t)n;
  uint32_t bits;
  if (exp2 == -14 && units < 1024) {
    bits = (uint32_t)units; /* subnormal (or zero) */
  } else {
    if (units == 2048) { /* rounded up to the next binade */
      units = 1024;
      exp2 += 1;
    }
    if (exp2 > 15) return (uint16_t)(sign | 0x7c00u);
    bits = ((uint32_t)(exp2 + 15) << 10) | (uint32_t)(units - 1024);
  }
  return (uint16_t)(sign | bits);
}

/* Round a double once to bfloat16 (1 sign, 8 exponent bits with bias 127, 7 fraction bits),
 * ties to even; returns the bit pattern.  Subnormals are multiples of 2^-133; values that
 * round to 2^128 or more overflow to infinity. */
uint16_t oracle_round_bf16(double x) {
  const uint16_t sign = signbit(x) ? 0x8000u : 0u;
  if (isnan(x)) return (uint16_t)(sign | 0x7fc0u);
  double a = fabs(x);
  if (isinf(a)) return (uint16_t)(sign | 0x7f80u);
  if (a == 0.0) return sign;
  int e;
  (void)frexp(a, &e);
  int exp2 = e - 1;
  if (exp2 < -126) exp2 = -126;
  const double q = ldexp(a, 7 - exp2); /* a in units of the spacing 2^(exp2-7); exact */
  uint64_t units = (uint64_t)nearbyint(q);
  uint32_t bits;
  if (exp2 == -126 && units < 128) {
    bits = (uint32_t)units;
  } else {
    if (units == 256) {
      units = 128;
      exp2 += 1;
    }
    if (exp2 > 127) return (uint16_t)(sign | 0x7f80u);
    bits = ((uint32_t)(exp2 + 127) << 7) | (uint32_t)(units - 128);
  }
  return (uint16_t)(sign | bits);
}

/* Packing (step 0 of the path; defined by the problem statement, not by the
 * paper): images are concatenated, each starting at the running byte count
 * rounded up to ORACLE_PACK_ALIGN; the total is rounded up too. */
int oracle_pack_size(const uint32_t* h, const uint32_t* w, uint32_t n, uint64_t* total) {
  if (!h || !w || !total || n == 0) return ORACLE_ERR_ARG;
  uint64_t at = 0;
  for (uint32_t i = 0; i < n; ++i) {
    if (h[i] == 0 || w[i] == 0) return ORACLE_ERR_ARG;
    at += (uint64_t)3 * h[i] * w[i];
    at = (at + ORACLE_PACK_ALIGN - 1) / ORACLE_PACK_ALIGN * ORACLE_PACK_ALIGN;
  }
  *total = at;
  return ORACLE_OK;
}

int oracle_pack(const uint8_t* const* images, const uint32_t* h, const uint32_t* w, uint32_t n,
                uint8_t* packed, uint64_t capacity, uint64_t* offsets) {
  uint64_t total;
  if (!images || !packed || !offsets) return ORACLE_ERR_ARG;
  if (oracle_pack_size(h, w, n, &total) != ORACLE_OK) return ORACLE_ERR_ARG;
  if (capacity < total) return ORACLE_ERR_SPACE;
  uint64_t at = 0;
  for (uint32_t i = 0; i < n; ++i) {
    if (!images[i]) return ORACLE_ERR_ARG;
    const uint64_t bytes = (uint64_t)3 * h[i] * w[i];
    offsets[i] = at;
    memcpy(packed + at, images[i], bytes);
    uint64_t end = at + bytes;
    uint64_t next = (end + ORACLE_PACK_ALIGN - 1) / ORACLE_PACK_ALIGN * ORACLE_PACK_ALIGN;
    memset(packed + end, 0, next - end);
    at = next;
  }
  return ORACLE_OK;
}

/* The whole batch: out is [n][3][c][c].  out_kind 0: double, 1: float (one
 * rounding from double), 2: binary16 bit patterns, 3: bfloat16 bit patterns (one
 * rounding from double each). */
typedef struct {
  const uint8_t* packed;
  const uint64_t* offsets;
  const uint32_t* h;
  const uint32_t* w;
  uint32_t first, last; /* images [first, last) */
  uint32_t c, s;
  const float* mean;
  const float* std;
  int out_kind;
  void* out;
  int rc;
} oracle_job_t;

static void oracle_store(void* out, int kind, size_t idx, double v) {
  if (kind == 0) ((double*)out)[idx] = v;
  else if (kind == 1) ((float*)out)[idx] = (float)v;
  else if (kind == 2) ((uint16_t*)out)[idx] = oracle_round_f16(v);
  else ((uint16_t*)out)[idx] = oracle_round_bf16(v);
}

static void* oracle_worker(void* arg) {
  oracle_job_t* job = (oracle_job_t*)arg;
  const uint32_t c = job->c;
  for (uint32_t i = job->first; i < job->last; ++i) {
    const uint8_t* img = job->packed + job->offsets[i];
    for (uint32_t ch = 0; ch < 3; ++ch)
      for (uint32_t k = 0; k < c; ++k)
        for (uint32_t j = 0; j < c; ++j) {
          double v;
          int rc = oracle_element(img, job->h[i], job->w[i], c, job->s, job->mean, job->std,
                                  ch, k, j, &v);
          if (rc != ORACLE_OK) {
            job->rc = rc;
            return NULL;
          }
          oracle_store(job->out, job->out_kind, (((size_t)i * 3 + ch) * c + k) * c + j, v);
        }
  }
  return NULL;
}

int oracle_preprocess(const uint8_t* packed, const uint64_t* offsets, const uint32_t* h,
                      const uint32_t* w, uint32_t n, uint32_t c, uint32_t s,
                      const float mean[3], const float std[3], int out_kind, void* out,
                      uint32_t nthreads) {
  if (!packed || !offsets || !h || !w || !mean || !std || !out || n == 0 || c == 0 || s < c)
    return ORACLE_ERR_ARG;
  if (out_kind < 0 || out_kind > 3) return ORACLE_ERR_ARG;
  for (int ch = 0; ch < 3; ++ch)
    if (!(std[ch] != 0.0f) || !isfinite(std[ch]) || !isfinite(mean[ch])) return ORACLE_ERR_ARG;
  for (uint32_t i = 0; i < n; ++i) {
    uint64_t rh, rw;
    if (oracle_resized_size(h[i], w[i], s, &rh, &rw) != ORACLE_OK) return ORACLE_ERR_ARG;
    if (rh < c || rw < c) return ORACLE_ERR_ARG;
  }
  if (nthreads == 0) nthreads = 1;
  if (nthreads > n) nthreads = n;
  oracle_job_t* jobs = (oracle_job_t*)calloc(nthreads, sizeof(oracle_job_t));
  pthread_t* tids = (pthread_t*)calloc(nthreads, sizeof(pthread_t));
  if (!jobs || !tids) {
    free(jobs);
    free(tids);
    return ORACLE_ERR_SPACE;
  }
  int rc = ORACLE_OK;
  for (uint32_t t = 0; t < nthreads; ++t) {
    jobs[t] = (oracle_job_t){packed, offsets, h, w,
                             (uint32_t)((uint64_t)n * t / nthreads),
                             (uint32_t)((uint64_t)n * (t + 1) / nthreads),
                             c, s, mean, std, out_kind, out, ORACLE_OK};
  }
  if (nthreads == 1) {
    oracle_worker(&jobs[0]);
  } else {
    for (uint32_t t = 0; t < nthreads; ++t) pthread_create(&tids[t], NULL, oracle_worker, &jobs[t]);
    for (uint32_t t = 0; t < nthreads; ++t) pthread_join(tids[t], NULL);
  }
  for (uint32_t t = 0; t < nthreads; ++t)
    if (jobs[t].rc != ORACLE_OK) rc = jobs[t].rc;
  free(jobs);
  free(tids);
  return rc;
}
