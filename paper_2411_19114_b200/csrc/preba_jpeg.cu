// JPEG Decode for a batch of baseline JPEG streams (sm_100a): the unit in front of Resize in the
// paper's image pipeline (Table 1 "Decode", Sec. 2.3 item 1, Sec. 4.2).  Baseline sequential DCT
// (ITU-T T.81: SOF0, 8-bit, Huffman, one interleaved scan, restart intervals), one or three
// components, luma sampled 1 or 2 times the chroma on each axis.
//
// The host reads the marker segments of every stream (a few hundred bytes each), writes one
// descriptor per image (sizes, sampling, quantisation tables, Huffman tables as MAXCODE / value
// offsets per code length plus an 8-bit look-up) and the entropy-coded bytes into a staging
// buffer, which is copied to the device once.  Three kernels follow on the stream:
//   find_segments   a block per image finds the restart markers of its scan, in order: the
//                   pieces between them decode independently;
//   decode_segments a thread per restart interval reads its bits (0xFF00 unstuffed), decodes the
//                   DC differences and AC runs of its MCUs and writes the quantised coefficients
//                   of every block in natural order (int16);
//   idct_colour     eight threads per 8 x 8 block, 32 blocks per CTA: dequantisation, the
//                   inverse DCT of T.81 A.3.3 in exact integers (the basis times 2^20, horizontal sums first and reduced by 2^9,
//                   vertical sums at scale 2^31, level shift, one rounding, clamp); chroma
//                   enlarged by replication; YCbCr -> RGB by the JFIF equations with the
//                   coefficients times 2^16 and one rounding; the pixels go straight into the
//                   packed HWC buffer and the {offset, h, w} table that preba_preprocess reads.
// Integer arithmetic throughout, so the decoded bytes are reproducible bit for bit.
#include <cuda_runtime.h>

#include <cstdint>
#include <cstring>

#include "preba.h"
#include "preba_internal.h"

namespace preba {
namespace jpeg {

constexpr uint32_t kMaxComp = 3;

// Figure A.6: the natural-order index of the k-th coded coefficient (one copy for the host's
// parser, one in device memory for the kernels).
#define PREBA_ZIGZAG_ORDER                                                                        \
  {0,  1,  8,  16, 9,  2,  3,  10, 17, 24, 32, 25, 18, 11, 4,  5,  12, 19, 26, 33, 40, 48,        \
   41, 34, 27, 20, 13, 6,  7,  14, 21, 28, 35, 42, 49, 56, 57, 50, 43, 36, 29, 22, 15, 23,        \
   30, 37, 44, 51, 58, 59, 52, 45, 38, 31, 39, 46, 53, 60, 61, 54, 47, 55, 62, 63}
static const uint8_t kZigzagHost[64] = PREBA_ZIGZAG_ORDER;
__device__ const uint8_t kZigzagDev[64] = PREBA_ZIGZAG_ORDER;

inline uint32_t zigzag(uint32_t k) { return kZigzagHost[k]; }

// One Huffman table as the decoder uses it (T.81 F.2.2.3): for code length l the largest code
// (maxcode, -1 if none) and the offset that turns a code into an index of vals; plus a look-up
// of the next 8 bits for the codes of up to 8 bits (length << 8 | value, 0: longer).
struct Huff {
  int32_t maxcode[18];
  int32_t valoff[18];
  uint16_t look[256];
  uint8_t vals[256];
};

struct Desc {
  uint64_t scan_off;   // of the entropy-coded bytes in the staging buffer
  uint64_t pix_off;    // of the image in the packed pixel buffer
  uint64_t coef_off;   // of the image's first block in the coefficient buffer, in blocks
  uint64_t seg_off;    // of the image's segment table in the staging buffer, in 4-byte units
  uint32_t scan_len;
  uint32_t w, h, ncomp;
  uint32_t hs[kMaxComp], vs[kMaxComp];   // sampling factors
  uint32_t hmax, vmax;
  uint32_t mcu_cols, mcu_rows;
  uint32_t ri;         // MCUs per restart interval (0: the scan is one piece)
  uint32_t nseg;       // pieces of the scan
  uint32_t comp_blocks[kMaxComp];        // blocks of component c before it, within the image
  uint16_t qt[kMaxComp][64];             // natural order
  Huff dc[kMaxComp], ac[kMaxComp];
};

// ---- the host's part: marker segments ----------------------------------------------------------------

struct Parsed {
  uint32_t w = 0, h = 0, ncomp = 0;
  uint32_t hs[kMaxComp] = {1, 1, 1}, vs[kMaxComp] = {1, 1, 1}, tq[kMaxComp] = {0, 0, 0};
  uint32_t td[kMaxComp] = {0, 0, 0}, ta[kMaxComp] = {0, 0, 0}, id[kMaxComp] = {0, 0, 0};
  uint32_t ri = 0;
  uint64_t scan_start = 0, scan_len = 0;
  bool have_qt[4] = {false, false, false, false};
  uint16_t qt[4][64];
  bool have_dc[4] = {false, false, false, false}, have_ac[4] = {false, false, false, false};
  uint8_t bits[2][4][16];
  uint8_t vals[2][4][256];
  uint32_t adobe_transform = 1;
};

// Reads the segments up to and including the scan header (T.81 B.2).
int parse(const uint8_t* d, uint64_t n, Parsed* p) {
  if (!d || n < 4 || d[0] != 0xFF || d[1] != 0xD8) return PREBA_ERR_BAD_STREAM;
  uint64_t at = 2;
  bool sof = false;
  for (;;) {
    if (at + 4 > n || d[at] != 0xFF) return PREBA_ERR_BAD_STREAM;
    while (at + 4 <= n && d[at + 1] == 0xFF) ++at;  // fill bytes
    if (at + 4 > n) return PREBA_ERR_BAD_STREAM;
    const uint32_t marker = d[at + 1];
    const uint64_t len = (static_cast<uint64_t>(d[at + 2]) << 8) | d[at + 3];
    if (len < 2 || at + 2 + len > n) return PREBA_ERR_BAD_STREAM;
    const uint8_t* seg = d + at + 4;
    const uint64_t sl = len - 2;
    if (marker == 0xDB) {  // DQT
      uint64_t k = 0;
      while (k < sl) {
        const uint32_t pq = seg[k] >> 4, tq = seg[k] & 15;
        ++k;
        const uint64_t cnt = pq ? 128 : 64;
        if (pq > 1 || tq > 3 || k + cnt > sl) return PREBA_ERR_BAD_STREAM;
        for (uint32_t z = 0; z < 64; ++z)
          p->qt[tq][zigzag(z)] = pq ? static_cast<uint16_t>((seg[k + 2 * z] << 8) | seg[k + 2 * z + 1])
                                    : seg[k + z];
        p->have_qt[tq] = true;
        k += cnt;
      }
    } else if (marker == 0xC4) {  // DHT
      uint64_t k = 0;
      while (k < sl) {
        if (k + 17 > sl) return PREBA_ERR_BAD_STREAM;
        const uint32_t tc = seg[k] >> 4, th = seg[k] & 15;
        uint32_t cnt = 0;
        for (uint32_t i = 0; i < 16; ++i) cnt += seg[k + 1 + i];
        if (tc > 1 || th > 3 || cnt > 256 || k + 17 + cnt > sl) return PREBA_ERR_BAD_STREAM;
        // code lengths must not be over-subscribed (Annex C)
        uint32_t code = 0;
        for (uint32_t l = 1; l <= 16; ++l) {
          code += seg[k + l];
          if (code > (1u << l)) return PREBA_ERR_BAD_STREAM;
          code <<= 1;
        }
        std::memcpy(p->bits[tc][th], seg + k + 1, 16);
        std::memset(p->vals[tc][th], 0, 256);
        std::memcpy(p->vals[tc][th], seg + k + 17, cnt);
        (tc ? p->have_ac : p->have_dc)[th] = true;
        k += 17 + cnt;
      }
    } else if (marker == 0xC0) {  // SOF0
      if (sof) return PREBA_ERR_UNSUPPORTED;
      sof = true;
      if (sl < 6) return PREBA_ERR_BAD_STREAM;
      if (seg[0] != 8) return PREBA_ERR_UNSUPPORTED;
      p->h = (seg[1] << 8) | seg[2];
      p->w = (seg[3] << 8) | seg[4];
      p->ncomp = seg[5];
      if (p->h == 0 || p->w == 0) return PREBA_ERR_UNSUPPORTED;  // size left to a DNL segment
      if ((p->ncomp != 1 && p->ncomp != 3) || sl != 6 + 3ull * p->ncomp) return PREBA_ERR_UNSUPPORTED;
      for (uint32_t i = 0; i < p->ncomp; ++i) {
        p->id[i] = seg[6 + 3 * i];
        p->hs[i] = seg[7 + 3 * i] >> 4;
        p->vs[i] = seg[7 + 3 * i] & 15;
        p->tq[i] = seg[8 + 3 * i];
        if (p->hs[i] < 1 || p->hs[i] > 2 || p->vs[i] < 1 || p->vs[i] > 2 || p->tq[i] > 3)
          return PREBA_ERR_UNSUPPORTED;
      }
      if (p->ncomp == 3 && (p->hs[1] != 1 || p->vs[1] != 1 || p->hs[2] != 1 || p->vs[2] != 1))
        return PREBA_ERR_UNSUPPORTED;
      if (p->ncomp == 1) p->hs[0] = p->vs[0] = 1;  // A.2.3: one block per MCU
    } else if ((marker >= 0xC1 && marker <= 0xCF && marker != 0xC4 && marker != 0xC8 &&
                marker != 0xCC)) {
      return PREBA_ERR_UNSUPPORTED;  // any frame type but baseline sequential DCT
    } else if (marker == 0xDD) {  // DRI
      if (sl < 2) return PREBA_ERR_BAD_STREAM;
      p->ri = (seg[0] << 8) | seg[1];
    } else if (marker == 0xEE && sl >= 12 && std::memcmp(seg, "Adobe", 5) == 0) {
      p->adobe_transform = seg[11];
    } else if (marker == 0xDA) {  // SOS
      if (!sof || sl < 1) return PREBA_ERR_BAD_STREAM;
      const uint32_t ns = seg[0];
      if (p->ncomp == 3 && p->adobe_transform == 0) return PREBA_ERR_UNSUPPORTED;
      if (ns != p->ncomp || sl != 4 + 2ull * ns) return PREBA_ERR_UNSUPPORTED;
      for (uint32_t j = 0; j < ns; ++j) {
        if (seg[1 + 2 * j] != p->id[j]) return PREBA_ERR_UNSUPPORTED;
        p->td[j] = seg[2 + 2 * j] >> 4;
        p->ta[j] = seg[2 + 2 * j] & 15;
        if (p->td[j] > 3 || p->ta[j] > 3) return PREBA_ERR_BAD_STREAM;
      }
      if (seg[1 + 2 * ns] != 0 || seg[2 + 2 * ns] != 63 || seg[3 + 2 * ns] != 0)
        return PREBA_ERR_UNSUPPORTED;
      for (uint32_t j = 0; j < ns; ++j)
        if (!p->have_qt[p->tq[j]] || !p->have_dc[p->td[j]] || !p->have_ac[p->ta[j]])
          return PREBA_ERR_BAD_STREAM;
      p->scan_start = at + 2 + len;
      p->scan_len = n - p->scan_start;
      return PREBA_OK;
    } else if (marker == 0xD9) {
      return PREBA_ERR_BAD_STREAM;  // end of image before any scan
    }
    at += 2 + len;
  }
}

void make_huff(const uint8_t bits[16], const uint8_t vals[256], Huff* t) {
  std::memset(t, 0, sizeof(*t));
  std::memcpy(t->vals, vals, 256);
  int32_t code = 0, at = 0;
  for (uint32_t l = 1; l <= 16; ++l) {
    const int32_t cnt = bits[l - 1];
    t->maxcode[l] = -1;
    if (cnt) {
      t->valoff[l] = at - code;  // index of a code of this length: code + valoff
      if (l <= 8)
        for (int32_t c = 0; c < cnt; ++c)
          for (uint32_t fill = 0; fill < (1u << (8 - l)); ++fill)
            t->look[((code + c) << (8 - l)) | fill] =
                static_cast<uint16_t>((l << 8) | vals[at + c]);
      code += cnt;
      t->maxcode[l] = code - 1;
      at += cnt;
    }
    code <<= 1;
  }
  t->maxcode[17] = 0x7fffffff;  // ends the search on a malformed stream
}

struct Layout {
  uint32_t mcu_cols, mcu_rows, hmax, vmax, nseg;
  uint64_t blocks;  // of the whole image
};

Layout layout_of(const Parsed& p) {
  Layout l;
  l.hmax = l.vmax = 1;
  for (uint32_t c = 0; c < p.ncomp; ++c) {
    l.hmax = p.hs[c] > l.hmax ? p.hs[c] : l.hmax;
    l.vmax = p.vs[c] > l.vmax ? p.vs[c] : l.vmax;
  }
  l.mcu_cols = (p.w + 8 * l.hmax - 1) / (8 * l.hmax);
  l.mcu_rows = (p.h + 8 * l.vmax - 1) / (8 * l.vmax);
  uint64_t per_mcu = 0;
  for (uint32_t c = 0; c < p.ncomp; ++c) per_mcu += p.hs[c] * p.vs[c];
  const uint64_t mcus = static_cast<uint64_t>(l.mcu_cols) * l.mcu_rows;
  l.blocks = mcus * per_mcu;
  l.nseg = p.ri ? static_cast<uint32_t>((mcus + p.ri - 1) / p.ri) : 1u;
  return l;
}

// ---- the device's part --------------------------------------------------------------------------------

struct Params {
  const uint8_t* stage;  // descriptors, then segment tables, then the scans
  int16_t* coef;
  uint8_t* pixels;
  int32_t* status;
  uint32_t n;
};

__device__ __forceinline__ const Desc& desc_of(const Params& p, uint32_t i) {
  return reinterpret_cast<const Desc*>(p.stage)[i];
}

__device__ __forceinline__ void report(int32_t* status, int code) {
  if (status) atomicCAS(status, 0, code);
}

// A block per image: seg[k] = first byte of piece k of the scan (seg[0] = 0), seg[nseg + k] =
// one past its last byte; pieces are separated by the restart markers, found in order.
__global__ void __launch_bounds__(256) find_segments(const Params p) {
  __shared__ uint32_t counts[256];
  __shared__ uint32_t found_total;
  const Desc& d = desc_of(p, blockIdx.x);
  uint32_t* seg = reinterpret_cast<uint32_t*>(const_cast<uint8_t*>(p.stage)) + d.seg_off;
  const uint8_t* scan = p.stage + d.scan_off;
  const uint32_t tid = threadIdx.x;
  if (d.ri == 0) {
    if (tid == 0) {
      seg[0] = 0;
      seg[1] = d.scan_len;
    }
    return;
  }
  const uint32_t chunk = (d.scan_len + 255u) / 256u;
  const uint32_t lo = tid * chunk, hi = min(d.scan_len, lo + chunk);
  uint32_t mine = 0;
  for (uint32_t i = lo; i < hi; ++i)
    if (scan[i] == 0xFF && i + 1 < d.scan_len && (scan[i + 1] & 0xF8) == 0xD0) ++mine;
  counts[tid] = mine;
  __syncthreads();
  if (tid == 0) {
    uint32_t run = 0;
    for (uint32_t t = 0; t < 256; ++t) {
      const uint32_t c = counts[t];
      counts[t] = run;
      run += c;
    }
    found_total = run;
    seg[0] = 0;
  }
  __syncthreads();
  const bool ok = found_total == d.nseg - 1;  // else the stream is damaged: decode nothing
  if (!ok) {
    if (tid == 0) {
      report(p.status, PREBA_ERR_BAD_STREAM);
      for (uint32_t k = 0; k < d.nseg; ++k) seg[k] = seg[d.nseg + k] = 0;
    }
    return;
  }
  uint32_t k = counts[tid];
  for (uint32_t i = lo; i < hi; ++i)
    if (scan[i] == 0xFF && i + 1 < d.scan_len && (scan[i + 1] & 0xF8) == 0xD0) {
      seg[d.nseg + k] = i;      // piece k ends in front of the marker
      seg[k + 1] = i + 2;       // piece k + 1 begins behind it
      ++k;
    }
  if (tid == 0) seg[2 * d.nseg - 1] = d.scan_len;
}

// The bits of one piece of a scan: a zero byte after 0xFF is stuffing; a marker, or the end of
// the piece, is followed by zeros.
struct BitReader {
  const uint8_t* at;
  const uint8_t* end;
  uint64_t acc;   // the next bits, left-aligned
  uint32_t have;  // valid bits in acc

  __device__ __forceinline__ void fill() {
    while (have <= 56) {
      uint32_t b = 0;
      if (at < end) {
        b = *at;
        if (b == 0xFF) {
          if (at + 1 < end && at[1] == 0) {
            at += 2;
          } else {
            at = end;  // a marker: nothing but zeros from here
            b = 0;
          }
        } else {
          ++at;
        }
      }
      acc |= static_cast<uint64_t>(b) << (56 - have);
      have += 8;
    }
  }
  __device__ __forceinline__ uint32_t peek(uint32_t n) const {
    return static_cast<uint32_t>(acc >> (64 - n));
  }
  __device__ __forceinline__ void skip(uint32_t n) {
    acc <<= n;
    have -= n;
  }
};

// One step of the decoder: DECODE (F.2.2.3, the 8-bit look-up in front) and, for a symbol that
// announces `size` further bits (all of a DC symbol, the low four bits of an AC symbol),
// RECEIVE and EXTEND (F.2.2.4, F.2.2.1), out of one 32-bit window of the stream: a code has at
// most 16 bits and a value at most 15.  Returns the symbol (256: no such code) and the value.
__device__ __forceinline__ uint32_t decode_step(BitReader& br, const Huff& t, bool dc, int32_t* value) {
  br.fill();
  const uint32_t w = br.peek(32);
  uint32_t len, sym;
  const uint32_t fast = t.look[w >> 24];
  if (fast) {
    len = fast >> 8;
    sym = fast & 0xffu;
  } else {
    len = 0;
    sym = 256u;
    for (uint32_t l = 9; l <= 16; ++l) {
      const int32_t code = static_cast<int32_t>(w >> (32 - l));
      if (code <= t.maxcode[l]) {
        len = l;
        sym = t.vals[(code + t.valoff[l]) & 255];
        break;
      }
    }
    if (sym > 255u) return sym;
  }
  const uint32_t size = dc ? sym : (sym & 15u);
  int32_t v = 0;
  if (size != 0 && size <= 15u) {
    v = static_cast<int32_t>((w << len) >> (32 - size));
    if (v < (1 << (size - 1))) v += 1 - (1 << size);
  }
  br.skip(len + (size <= 15u ? size : 0u));
  *value = v;
  return sym;
}

// A thread per piece of a scan (blockIdx.y: image).  Writes the quantised coefficients of its
// MCUs' blocks, natural order, into the zeroed coefficient buffer: per MCU the blocks of
// component 0, then 1, then 2, each in raster order inside the MCU.
#ifndef PREBA_JPEG_LANES
#define PREBA_JPEG_LANES 4
#endif
// Lanes of a warp that decode (the others idle): lanes in different places of the decoding
// loops run in turn, so a warp with few of them wastes little, and more warps keep the
// schedulers busy while each waits for its own chain of dependent instructions.
constexpr uint32_t kDecodeLanes = PREBA_JPEG_LANES;
constexpr uint32_t kDecodeThreads = 128;
constexpr uint32_t kDecodePerBlock = kDecodeThreads / 32 * kDecodeLanes;

__global__ void __launch_bounds__(kDecodeThreads) decode_segments(const Params p) {
  const Desc& d = desc_of(p, blockIdx.y);
  if ((threadIdx.x & 31u) >= kDecodeLanes) return;
  const uint32_t s = blockIdx.x * kDecodePerBlock + (threadIdx.x >> 5) * kDecodeLanes + (threadIdx.x & 31u);
  if (s >= d.nseg) return;
  const uint32_t* seg = reinterpret_cast<const uint32_t*>(p.stage) + d.seg_off;
  const uint32_t lo = seg[s], hi = seg[d.nseg + s];
  if (hi <= lo || hi > d.scan_len) return;  // an empty or damaged piece: its blocks stay zero
  BitReader br;
  br.at = p.stage + d.scan_off + lo;
  br.end = p.stage + d.scan_off + hi;
  br.acc = 0;
  br.have = 0;
  const uint32_t mcus = d.mcu_cols * d.mcu_rows;
  const uint32_t first = d.ri ? s * d.ri : 0u;
  const uint32_t last = d.ri ? min(mcus, first + d.ri) : mcus;
  uint32_t per_mcu = 0;
  for (uint32_t c = 0; c < d.ncomp; ++c) per_mcu += d.hs[c] * d.vs[c];
  int32_t pred[kMaxComp] = {0, 0, 0};
  for (uint32_t m = first; m < last; ++m) {
    int16_t* block = p.coef + (d.coef_off + static_cast<uint64_t>(m) * per_mcu) * 64;
    for (uint32_t c = 0; c < d.ncomp; ++c) {
      const Huff& dc = d.dc[c];
      const Huff& ac = d.ac[c];
      for (uint32_t b = 0; b < d.hs[c] * d.vs[c]; ++b, block += 64) {
        int32_t v;
        const uint32_t t = decode_step(br, dc, true, &v);
        if (t > 11) {
          report(p.status, PREBA_ERR_BAD_STREAM);
          return;
        }
        pred[c] += v;
        block[0] = static_cast<int16_t>(pred[c]);
        for (uint32_t k = 1; k < 64;) {
          const uint32_t rs = decode_step(br, ac, false, &v);
          if (rs > 255) {
            report(p.status, PREBA_ERR_BAD_STREAM);
            return;
          }
          const uint32_t run = rs >> 4, size = rs & 15;
          if (size == 0) {
            if (run != 15) break;  // EOB
            k += 16;               // ZRL
            continue;
          }
          k += run;
          if (k > 63) {
            report(p.status, PREBA_ERR_BAD_STREAM);
            return;
          }
          block[kZigzagDev[k]] = static_cast<int16_t>(v);
          ++k;
        }
      }
    }
  }
}

// round(2^20 (C_u / 2) cos((2x + 1) u pi / 16)) of T.81 A.3.3, from round(2^20 cos(k pi / 16) / 2),
// k = 0..7, by symmetry; a compile-time constant wherever x and u are.
__host__ __device__ constexpr int32_t cos_fix(uint32_t k) {
  return k == 0 ? 524288 : k == 1 ? 514214 : k == 2 ? 484379 : k == 3 ? 435930 : k == 4 ? 370728
         : k == 5 ? 291279 : k == 6 ? 200636 : 102284;
}
__host__ __device__ constexpr int32_t basis(uint32_t x, uint32_t u) {
  if (u == 0) return cos_fix(4);
  uint32_t k = ((2 * x + 1) * u) & 31u;
  if (k > 16) k = 32 - k;
  return k <= 7 ? cos_fix(k) : (k == 8 ? 0 : -cos_fix(16 - k));
}

// The eight sums sum_u basis(x, u) in[u], x = 0..7, exact in 64 bits.  basis(7 - x, u) is
// basis(x, u) for even u and its negative for odd u, so the even and the odd terms are summed
// once for x and 7 - x.
__device__ __forceinline__ void transform8(const int32_t (&in)[8], int64_t (&out)[8]) {
#pragma unroll
  for (uint32_t x = 0; x < 4; ++x) {
    int64_t even = 0, odd = 0;
#pragma unroll
    for (uint32_t u = 0; u < 8; u += 2) {
      even += static_cast<int64_t>(basis(x, u)) * in[u];
      odd += static_cast<int64_t>(basis(x, u + 1)) * in[u + 1];
    }
    out[x] = even + odd;
    out[7 - x] = even - odd;
  }
}

__device__ __forceinline__ uint32_t clamp255(int32_t v) {
  return v <= 0 ? 0u : (v >= 255 ? 255u : static_cast<uint32_t>(v));
}

// Eight threads per 8 x 8 block, 32 blocks per CTA: as many whole MCUs as that holds
// (blockIdx.y: image).  A thread takes a row of the block through the horizontal sums, then,
// after an exchange through shared memory within its warp, a column through the vertical
// ones; then all threads convert the MCUs' pixels and store them.  Exact integer arithmetic
// throughout: the basis times 2^20, the row sums reduced by 2^9, the column sums at scale 2^31.
constexpr uint32_t kIdctThreads = 256;
constexpr uint32_t kIdctBlocks = kIdctThreads / 8;
constexpr uint32_t kTilePitch = 72;  // words between the blocks' tiles: four blocks of a warp
                                     // read eight words each from different banks

__host__ __device__ inline uint32_t mcus_per_cta(uint32_t blocks_per_mcu) {
  return kIdctBlocks / blocks_per_mcu;
}

__global__ void __launch_bounds__(kIdctThreads) idct_colour(const Params p) {
  __shared__ __align__(16) int32_t tile[kIdctBlocks * kTilePitch];  // row sums, [v][x] per block
  __shared__ uint8_t smp[kIdctBlocks][64];                           // the samples of the blocks
  const Desc& d = desc_of(p, blockIdx.y);
  const uint32_t mcus = d.mcu_cols * d.mcu_rows;
  uint32_t per_mcu = 0;
  for (uint32_t c = 0; c < d.ncomp; ++c) per_mcu += d.hs[c] * d.vs[c];
  const uint32_t held = mcus_per_cta(per_mcu), first = blockIdx.x * held;
  if (first >= mcus) return;
  const uint32_t tid = threadIdx.x, group = tid >> 3, r = tid & 7u;
  const uint32_t local = group / per_mcu, blk = group - local * per_mcu, mcu = first + local;
  const bool live = local < held && mcu < mcus;
  if (live) {
    uint32_t comp = 0, before = 0;
    while (comp + 1 < d.ncomp && blk >= before + d.hs[comp] * d.vs[comp]) {
      before += d.hs[comp] * d.vs[comp];
      ++comp;
    }
    // row r of the block: S = Sq * Q (A.3.4), limited to what the sums below hold (a valid
    // stream stays far inside)
    const int16_t* coef = p.coef + (d.coef_off + static_cast<uint64_t>(mcu) * per_mcu + blk) * 64 + 8u * r;
    const int4 raw = *reinterpret_cast<const int4*>(coef);
    const int32_t packed[4] = {raw.x, raw.y, raw.z, raw.w};
    const uint16_t* q = d.qt[comp] + 8u * r;
    int32_t in[8];
#pragma unroll
    for (uint32_t u = 0; u < 8; ++u) {
      const int32_t c16 = static_cast<int16_t>(static_cast<uint32_t>(packed[u >> 1]) >> (16u * (u & 1u)));
      in[u] = max(-16383, min(16383, c16 * static_cast<int32_t>(q[u])));
    }
    int64_t t[8];
    transform8(in, t);
    int32_t* row = tile + group * kTilePitch + 8u * r;
#pragma unroll
    for (uint32_t x = 0; x < 8; ++x) row[x] = static_cast<int32_t>((t[x] + (1 << 8)) >> 9);
  }
  __syncwarp();  // the eight threads of a block are in one warp
  if (live) {
    // column r of the block
    int32_t in[8];
#pragma unroll
    for (uint32_t v = 0; v < 8; ++v) in[v] = tile[group * kTilePitch + 8u * v + r];
    int64_t sum[8];
    transform8(in, sum);
#pragma unroll
    for (uint32_t y = 0; y < 8; ++y)
      smp[group][8u * y + r] = static_cast<uint8_t>(
          clamp255(static_cast<int32_t>((sum[y] + (128ll << 31) + (1ll << 30)) >> 31)));
  }
  __syncthreads();
  // the MCUs' pixels: 8 hmax x 8 vmax each (hmax, vmax are 1 or 2); a chroma sample serves
  // hmax x vmax of them
  const uint32_t xs = d.hmax >> 1, ys_ = d.vmax >> 1;          // shifts: log2 of hmax, vmax
  const uint32_t mw_log = 3u + xs, px_log = 6u + xs + ys_;       // log2 of the MCU's width, pixels
  const uint32_t here = min(held, mcus - first);
  const uint32_t nluma = d.hs[0] * d.vs[0];
  uint8_t* img = p.pixels + d.pix_off;
  for (uint32_t i = tid; i < (here << px_log); i += kIdctThreads) {
    const uint32_t loc = i >> px_log, within = i & ((1u << px_log) - 1u);
    const uint32_t py = within >> mw_log, px = within & ((1u << mw_log) - 1u);
    const uint32_t m = first + loc;
    const uint32_t my = m / d.mcu_cols, mx = m - my * d.mcu_cols;
    const uint32_t gy = (my << (3u + ys_)) + py, gx = (mx << mw_log) + px;
    if (gy >= d.h || gx >= d.w) continue;
    const uint32_t base = loc * per_mcu;
    // the luma block that holds the pixel (raster order inside the MCU)
    const uint32_t ys = smp[base + (py >> 3) * d.hs[0] + (px >> 3)][8u * (py & 7u) + (px & 7u)];
    uint32_t red = ys, green = ys, blue = ys;
    if (d.ncomp == 3) {
      const uint32_t at = 8u * (py >> ys_) + (px >> xs);  // chroma sampled once per MCU block
      const int32_t y16 = static_cast<int32_t>(ys << 16) + (1 << 15);
      const int32_t cb = static_cast<int32_t>(smp[base + nluma][at]) - 128;
      const int32_t cr = static_cast<int32_t>(smp[base + nluma + 1][at]) - 128;
      // the JFIF coefficients as round(2^16 c); one rounding each
      red = clamp255((y16 + 91881 * cr) >> 16);
      green = clamp255((y16 - 22553 * cb - 46802 * cr) >> 16);
      blue = clamp255((y16 + 116130 * cb) >> 16);
    }
    uint8_t* out = img + 3ull * (static_cast<uint64_t>(gy) * d.w + gx);
    out[0] = static_cast<uint8_t>(red);
    out[1] = static_cast<uint8_t>(green);
    out[2] = static_cast<uint8_t>(blue);
  }
}

uint64_t stage_header_bytes(uint32_t n) { return align_up(static_cast<uint64_t>(n) * sizeof(Desc), 256); }

}  // namespace jpeg
}  // namespace preba

extern "C" int preba_jpeg_query(const uint8_t* const* jpegs, const uint64_t* bytes, uint32_t n,
                                uint32_t* h, uint32_t* w, preba_jpeg_sizes_t* sizes) {
  using namespace preba;
  using namespace preba::jpeg;
  if (!jpegs || !bytes || !sizes || n == 0) return PREBA_ERR_INVALID_ARG;
  uint64_t stage = stage_header_bytes(n), segs = 0, scans = 0, blocks = 0, packed = 0;
  for (uint32_t i = 0; i < n; ++i) {
    Parsed p;
    const int rc = parse(jpegs[i], bytes[i], &p);
    if (rc != PREBA_OK) return rc;
    if (p.w > PREBA_MAX_DIM || p.h > PREBA_MAX_DIM || p.scan_len > 0xfffffff0ull)
      return PREBA_ERR_UNSUPPORTED;
    const Layout l = layout_of(p);
    if (h) h[i] = p.h;
    if (w) w[i] = p.w;
    segs += 2ull * l.nseg;
    scans += align_up(p.scan_len, 16);
    blocks += l.blocks;
    packed = align_up(packed + 3ull * p.h * p.w, PREBA_PACK_ALIGN);
  }
  sizes->stage_bytes = stage + align_up(4 * segs, 256) + scans;
  sizes->coef_bytes = blocks * 64 * sizeof(int16_t);
  sizes->packed_bytes = packed;
  sizes->table_bytes = static_cast<uint64_t>(n) * sizeof(preba_img_t);
  return PREBA_OK;
}

extern "C" int preba_jpeg_decode(const preba_jpeg_batch_t* b, void* stream) {
  using namespace preba;
  using namespace preba::jpeg;
  if (!b || !b->jpegs || !b->bytes || b->n == 0 || !b->stage_host || !b->stage_dev || !b->coef ||
      !b->pixels || !b->table || !b->table_host || b->n > 65535u)
    return PREBA_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(b->stage_dev) % 16 || reinterpret_cast<uintptr_t>(b->stage_host) % 16 ||
      reinterpret_cast<uintptr_t>(b->pixels) % 16 || reinterpret_cast<uintptr_t>(b->coef) % 16 ||
      reinterpret_cast<uintptr_t>(b->table) % 8)
    return PREBA_ERR_INVALID_ARG;
  // pass 1: sizes (segment tables come before the scans)
  uint64_t segs = 0;
  uint32_t most_seg = 1, most_mcus = 1;
  for (uint32_t i = 0; i < b->n; ++i) {
    Parsed p;
    const int rc = parse(b->jpegs[i], b->bytes[i], &p);
    if (rc != PREBA_OK) return rc;
    if (p.w > PREBA_MAX_DIM || p.h > PREBA_MAX_DIM || p.scan_len > 0xfffffff0ull)
      return PREBA_ERR_UNSUPPORTED;
    segs += 2ull * layout_of(p).nseg;
  }
  const uint64_t seg_base = stage_header_bytes(b->n);
  uint64_t at_seg = 0, at_scan = seg_base + align_up(4 * segs, 256), at_block = 0, at_pix = 0;
  Desc* descs = reinterpret_cast<Desc*>(b->stage_host);
  for (uint32_t i = 0; i < b->n; ++i) {
    Parsed p;
    (void)parse(b->jpegs[i], b->bytes[i], &p);
    const Layout l = layout_of(p);
    if (at_scan + align_up(p.scan_len, 16) > b->stage_bytes) return PREBA_ERR_BUFFER_TOO_SMALL;
    Desc& d = descs[i];
    std::memset(&d, 0, sizeof(d));
    d.scan_off = at_scan;
    d.scan_len = static_cast<uint32_t>(p.scan_len);
    d.pix_off = at_pix;
    d.coef_off = at_block;
    d.seg_off = seg_base / 4 + at_seg;
    d.w = p.w;
    d.h = p.h;
    d.ncomp = p.ncomp;
    d.hmax = l.hmax;
    d.vmax = l.vmax;
    d.mcu_cols = l.mcu_cols;
    d.mcu_rows = l.mcu_rows;
    d.ri = p.ri;
    d.nseg = l.nseg;
    uint32_t before = 0;
    for (uint32_t c = 0; c < p.ncomp; ++c) {
      d.hs[c] = p.hs[c];
      d.vs[c] = p.vs[c];
      d.comp_blocks[c] = before;
      before += p.hs[c] * p.vs[c];
      std::memcpy(d.qt[c], p.qt[p.tq[c]], sizeof(d.qt[c]));
      make_huff(p.bits[0][p.td[c]], p.vals[0][p.td[c]], &d.dc[c]);
      make_huff(p.bits[1][p.ta[c]], p.vals[1][p.ta[c]], &d.ac[c]);
    }
    std::memcpy(b->stage_host + at_scan, b->jpegs[i] + p.scan_start, p.scan_len);
    std::memset(b->stage_host + at_scan + p.scan_len, 0, align_up(p.scan_len, 16) - p.scan_len);
    b->table_host[i].offset = at_pix;
    b->table_host[i].h = p.h;
    b->table_host[i].w = p.w;
    most_seg = l.nseg > most_seg ? l.nseg : most_seg;
    // CTAs of the inverse transform: as many whole MCUs each as its 32 blocks hold
    const uint32_t mcus = l.mcu_cols * l.mcu_rows, held = mcus_per_cta(before);
    most_mcus = (mcus + held - 1) / held > most_mcus ? (mcus + held - 1) / held : most_mcus;
    at_seg += 2ull * l.nseg;
    at_scan += align_up(p.scan_len, 16);
    at_block += l.blocks;
    at_pix = align_up(at_pix + 3ull * p.h * p.w, PREBA_PACK_ALIGN);
  }
  if (at_block * 128 > b->coef_bytes || at_pix > b->pixels_bytes) return PREBA_ERR_BUFFER_TOO_SMALL;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  cudaError_t err = cudaMemcpyAsync(b->stage_dev, b->stage_host, at_scan, cudaMemcpyHostToDevice, s);
  if (err == cudaSuccess)
    err = cudaMemcpyAsync(b->table, b->table_host, sizeof(preba_img_t) * b->n,
                          cudaMemcpyHostToDevice, s);
  if (err == cudaSuccess) err = cudaMemsetAsync(b->coef, 0, at_block * 128, s);
  if (err == cudaSuccess) {
    Params p;
    p.stage = b->stage_dev;
    p.coef = b->coef;
    p.pixels = b->pixels;
    p.status = b->status;
    p.n = b->n;
    find_segments<<<b->n, 256, 0, s>>>(p);
    decode_segments<<<dim3((most_seg + kDecodePerBlock - 1) / kDecodePerBlock, b->n), kDecodeThreads, 0, s>>>(p);
    idct_colour<<<dim3(most_mcus, b->n), kIdctThreads, 0, s>>>(p);
    err = cudaGetLastError();
  }
  if (err != cudaSuccess) {
    g_last_cuda_error = static_cast<int>(err);
    return PREBA_ERR_CUDA;
  }
  return PREBA_OK;
}
