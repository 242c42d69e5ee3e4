/*
 * TEST INFRASTRUCTURE ONLY — CPU oracle for the variants of the vision preprocessing path:
 * an explicit crop origin per image, and a resize whose result is rounded to uint8.
 *
 * The paper names the operations (Resize, Crop, Normalize; Sec. 2.3 item 1, Table 1) and says
 * that other models need "only incremental adjustments" of the same units (Sec. 4.2, "Flexible
 * design based on reconfigurable hardware"); it fixes none of the numerics.  The readings
 * taken here, beside those of the base oracle (same sampling geometry, same resized size):
 *   - crop origin: the window's first row and column on the resized grid, (top, left), given
 *     per image, with top + c <= R_h and left + c <= R_w; the centre crop is the special case
 *     (floor((R_h - c)/2), floor((R_w - c)/2));
 *   - rounding to uint8: the bilinear value v is a ratio of integers (weights are rem/den per
 *     axis), and the rounded pixel is floor(v + 1/2), decided in exact integer arithmetic:
 *     floor((2*num + den) / (2*den)).  Ties go up.  No clamp is needed (0 <= v <= 255);
 *   - uint8 output: the rounded pixels of the crop window, HWC, [n][c][c][3], no normalisation;
 *   - float output after rounding: ((q/255) - mean_c)/std_c on the rounded pixel q, planar.
 *
 * It shares nothing with the CUDA path and nothing with the base oracle's source file; only
 * tests, the smoke check and the benchmark's CPU legs call it.  Every function is pinned by
 * tests that do not use it to make their expected values (identity, pure crop at an explicit
 * origin, constant images, ramps with known ties, exact-rational brute force, sub-windows of
 * the base oracle's output): none is "parity unpinned".
 */
#include <math.h>
#include <pthread.h>
#include <stdint.h>
#include <stdlib.h>

#define VAR_OK 0
#define VAR_ERR_ARG -1
#define VAR_ERR_SPACE -2

typedef unsigned __int128 u128;

/* Resized size: shorter side -> s, longer -> floor(s*long/short) (as the base path). */
static void var_resized(uint32_t h, uint32_t w, uint32_t s, uint64_t* rh, uint64_t* rw) {
  if (h <= w) {
    *rh = s;
    *rw = ((uint64_t)s * w) / h;
  } else {
    *rw = s;
    *rh = ((uint64_t)s * h) / w;
  }
}

/* One axis: resized index X = origin + j samples source coordinate (X + 1/2)*in/r - 1/2
 * clamped to [0, in-1] = num/den with num = (2X+1)*in - r, den = 2r.  Returns the taps, the
 * remainder (weight of the second tap is rem/den) and den. */
int oracle_var_axis(uint32_t in, uint64_t r, uint64_t origin, uint32_t j, uint32_t* i0,
                    uint32_t* i1, uint64_t* rem, uint64_t* den) {
  if (in == 0 || r == 0 || origin + j >= r || !i0 || !i1 || !rem || !den) return VAR_ERR_ARG;
  const uint64_t X = origin + j;
  const int64_t d = 2 * (int64_t)r;
  int64_t num = (2 * (int64_t)X + 1) * (int64_t)in - (int64_t)r;
  const int64_t hi = ((int64_t)in - 1) * d;
  if (num < 0) num = 0;
  if (num > hi) num = hi;
  const int64_t q = num / d;
  *i0 = (uint32_t)q;
  *i1 = (uint32_t)((q + 1 < (int64_t)in) ? q + 1 : (int64_t)in - 1);
  *rem = (uint64_t)(num % d);
  *den = (uint64_t)d;
  return VAR_OK;
}

/* The four taps and the two weights of output (k, j) of one image for a window at (top, left). */
typedef struct {
  uint32_t x0, x1, y0, y1;
  uint64_t rx, dx, ry, dy;
} var_taps_t;

static int var_taps(uint32_t h, uint32_t w, uint32_t c, uint32_t s, uint64_t top, uint64_t left,
                    uint32_t k, uint32_t j, var_taps_t* t) {
  uint64_t rh, rw;
  if (h == 0 || w == 0 || s == 0 || c == 0 || k >= c || j >= c) return VAR_ERR_ARG;
  var_resized(h, w, s, &rh, &rw);
  if (top + c > rh || left + c > rw) return VAR_ERR_ARG;
  if (oracle_var_axis(w, rw, left, j, &t->x0, &t->x1, &t->rx, &t->dx) != VAR_OK) return VAR_ERR_ARG;
  if (oracle_var_axis(h, rh, top, k, &t->y0, &t->y1, &t->ry, &t->dy) != VAR_OK) return VAR_ERR_ARG;
  return VAR_OK;
}

/* The bilinear value of channel ch at output (k, j), unrounded, in double, difference form
 * (as the base path computes it), for a window at (top, left). */
int oracle_var_value(const uint8_t* img, uint32_t h, uint32_t w, uint32_t c, uint32_t s,
                     uint64_t top, uint64_t left, uint32_t ch, uint32_t k, uint32_t j,
                     double* v) {
  var_taps_t t;
  if (!img || !v || ch > 2) return VAR_ERR_ARG;
  if (var_taps(h, w, c, s, top, left, k, j, &t) != VAR_OK) return VAR_ERR_ARG;
  const size_t pitch = (size_t)3 * w;
  const double p00 = img[t.y0 * pitch + 3 * (size_t)t.x0 + ch];
  const double p01 = img[t.y0 * pitch + 3 * (size_t)t.x1 + ch];
  const double p10 = img[t.y1 * pitch + 3 * (size_t)t.x0 + ch];
  const double p11 = img[t.y1 * pitch + 3 * (size_t)t.x1 + ch];
  const double lx = (double)t.rx / (double)t.dx, ly = (double)t.ry / (double)t.dy;
  const double a = p00 + lx * (p01 - p00);
  const double b = p10 + lx * (p11 - p10);
  *v = a + ly * (b - a);
  return VAR_OK;
}

/* The same value rounded to the nearest integer, ties up, decided exactly:
 * v = num / (dx*dy) with num = (p00*(dx-rx) + p01*rx)*(dy-ry) + (p10*(dx-rx) + p11*rx)*ry,
 * q = floor((2*num + dx*dy) / (2*dx*dy)). */
int oracle_var_pixel_u8(const uint8_t* img, uint32_t h, uint32_t w, uint32_t c, uint32_t s,
                        uint64_t top, uint64_t left, uint32_t ch, uint32_t k, uint32_t j,
                        uint8_t* q) {
  var_taps_t t;
  if (!img || !q || ch > 2) return VAR_ERR_ARG;
  if (var_taps(h, w, c, s, top, left, k, j, &t) != VAR_OK) return VAR_ERR_ARG;
  const size_t pitch = (size_t)3 * w;
  const u128 p00 = img[t.y0 * pitch + 3 * (size_t)t.x0 + ch];
  const u128 p01 = img[t.y0 * pitch + 3 * (size_t)t.x1 + ch];
  const u128 p10 = img[t.y1 * pitch + 3 * (size_t)t.x0 + ch];
  const u128 p11 = img[t.y1 * pitch + 3 * (size_t)t.x1 + ch];
  const u128 upper = p00 * (t.dx - t.rx) + p01 * t.rx;
  const u128 lower = p10 * (t.dx - t.rx) + p11 * t.rx;
  const u128 num = upper * (t.dy - t.ry) + lower * t.ry;
  const u128 den = (u128)t.dx * t.dy;
  *q = (uint8_t)((2 * num + den) / (2 * den));
  return VAR_OK;
}

/* IEEE binary16 / bfloat16 roundings of the float outputs, ties to even, written from the
 * formats (1+5+10 bits, bias 15; 1+8+7 bits, bias 127); subnormals and overflow handled. */
static uint16_t var_round_small(double x, int frac_bits, int min_exp, int max_exp, int bias,
                                uint16_t inf_bits, uint16_t nan_bits) {
  const uint16_t sign = signbit(x) ? 0x8000u : 0u;
  if (isnan(x)) return (uint16_t)(sign | nan_bits);
  double a = fabs(x);
  if (isinf(a)) return (uint16_t)(sign | inf_bits);
  if (a == 0.0) return sign;
  int e;
  (void)frexp(a, &e);
  int exp2 = e - 1;
  if (exp2 < min_exp) exp2 = min_exp;
  const uint64_t one = (uint64_t)1 << frac_bits;
  uint64_t units = (uint64_t)nearbyint(ldexp(a, frac_bits - exp2));
  if (exp2 == min_exp && units < one) return (uint16_t)(sign | units);
  if (units == 2 * one) {
    units = one;
    exp2 += 1;
  }
  if (exp2 > max_exp) return (uint16_t)(sign | inf_bits);
  return (uint16_t)(sign | ((uint32_t)(exp2 + bias) << frac_bits) | (uint32_t)(units - one));
}

/* The whole batch.
 *   crop_origin  NULL (centre crop) or 2n values (top, left) per image
 *   round_u8     0: normalise the unrounded value; 1: round to uint8 first
 *   out_kind     0 double, 1 float, 2 binary16 bits, 3 bfloat16 bits: planar [n][3][c][c],
 *                out = (v/255 - mean)/std;  4: uint8 HWC [n][c][c][3], the rounded pixel itself
 *                (requires round_u8) */
typedef struct {
  const uint8_t* packed;
  const uint64_t* offsets;
  const uint32_t* h;
  const uint32_t* w;
  uint32_t first, last;
  uint32_t c, s;
  const float* mean;
  const float* std;
  const uint32_t* crop_origin;
  int round_u8, out_kind;
  void* out;
  int rc;
} var_job_t;

static void* var_worker(void* arg) {
  var_job_t* job = (var_job_t*)arg;
  const uint32_t c = job->c;
  for (uint32_t i = job->first; i < job->last; ++i) {
    const uint8_t* img = job->packed + job->offsets[i];
    uint64_t rh, rw;
    var_resized(job->h[i], job->w[i], job->s, &rh, &rw);
    const uint64_t top = job->crop_origin ? job->crop_origin[2 * i] : (rh - c) / 2;
    const uint64_t left = job->crop_origin ? job->crop_origin[2 * i + 1] : (rw - c) / 2;
    for (uint32_t ch = 0; ch < 3; ++ch)
      for (uint32_t k = 0; k < c; ++k)
        for (uint32_t j = 0; j < c; ++j) {
          double v = 0.0;
          uint8_t q = 0;
          const int rc = job->round_u8
              ? oracle_var_pixel_u8(img, job->h[i], job->w[i], c, job->s, top, left, ch, k, j, &q)
              : oracle_var_value(img, job->h[i], job->w[i], c, job->s, top, left, ch, k, j, &v);
          if (rc != VAR_OK) {
            job->rc = rc;
            return NULL;
          }
          if (job->out_kind == 4) {
            ((uint8_t*)job->out)[(((size_t)i * c + k) * c + j) * 3 + ch] = q;
            continue;
          }
          if (job->round_u8) v = q;
          const double o = (v / 255.0 - (double)job->mean[ch]) / (double)job->std[ch];
          const size_t idx = (((size_t)i * 3 + ch) * c + k) * c + j;
          if (job->out_kind == 0) ((double*)job->out)[idx] = o;
          else if (job->out_kind == 1) ((float*)job->out)[idx] = (float)o;
          else if (job->out_kind == 2)
            ((uint16_t*)job->out)[idx] = var_round_small(o, 10, -14, 15, 15, 0x7c00u, 0x7e00u);
          else
            ((uint16_t*)job->out)[idx] = var_round_small(o, 7, -126, 127, 127, 0x7f80u, 0x7fc0u);
        }
  }
  return NULL;
}

int oracle_var_preprocess(const uint8_t* packed, const uint64_t* offsets, const uint32_t* h,
                          const uint32_t* w, uint32_t n, uint32_t c, uint32_t s,
                          const float mean[3], const float std[3], const uint32_t* crop_origin,
                          int round_u8, int out_kind, void* out, uint32_t nthreads) {
  if (!packed || !offsets || !h || !w || !out || n == 0 || c == 0 || s < c) return VAR_ERR_ARG;
  if (out_kind < 0 || out_kind > 4 || (out_kind == 4 && !round_u8)) return VAR_ERR_ARG;
  if (out_kind != 4) {
    if (!mean || !std) return VAR_ERR_ARG;
    for (int ch = 0; ch < 3; ++ch)
      if (!(std[ch] != 0.0f) || !isfinite(std[ch]) || !isfinite(mean[ch])) return VAR_ERR_ARG;
  }
  for (uint32_t i = 0; i < n; ++i) {
    uint64_t rh, rw;
    if (h[i] == 0 || w[i] == 0) return VAR_ERR_ARG;
    var_resized(h[i], w[i], s, &rh, &rw);
    if (rh < c || rw < c) return VAR_ERR_ARG;
    if (crop_origin && ((uint64_t)crop_origin[2 * i] + c > rh ||
                        (uint64_t)crop_origin[2 * i + 1] + c > rw))
      return VAR_ERR_ARG;
  }
  if (nthreads == 0) nthreads = 1;
  if (nthreads > n) nthreads = n;
  var_job_t* jobs = (var_job_t*)calloc(nthreads, sizeof(var_job_t));
  pthread_t* tids = (pthread_t*)calloc(nthreads, sizeof(pthread_t));
  if (!jobs || !tids) {
    free(jobs);
    free(tids);
    return VAR_ERR_SPACE;
  }
  for (uint32_t t = 0; t < nthreads; ++t)
    jobs[t] = (var_job_t){packed, offsets, h, w,
                          (uint32_t)((uint64_t)n * t / nthreads),
                          (uint32_t)((uint64_t)n * (t + 1) / nthreads),
                          c, s, mean, std, crop_origin, round_u8, out_kind, out, VAR_OK};
  if (nthreads == 1) {
    var_worker(&jobs[0]);
  } else {
    for (uint32_t t = 0; t < nthreads; ++t) pthread_create(&tids[t], NULL, var_worker, &jobs[t]);
    for (uint32_t t = 0; t < nthreads; ++t) pthread_join(tids[t], NULL);
  }
  int rc = VAR_OK;
  for (uint32_t t = 0; t < nthreads; ++t)
    if (jobs[t].rc != VAR_OK) rc = jobs[t].rc;
  free(jobs);
  free(tids);
  return rc;
}
