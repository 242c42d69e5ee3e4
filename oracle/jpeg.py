"""TEST INFRASTRUCTURE ONLY: CPU oracle of the JPEG Decode unit (plain Python and numpy).

The paper's image pipeline starts with "Decode" (Table 1, the largest image unit of the DPU;
Sec. 2.3 item 1: JPEG to RGB; Sec. 4.2: Decode -> Resize -> Crop -> Normalize chained on chip).
It names no numerics.  This file decodes baseline sequential JPEG (ITU-T T.81 / ISO 10918-1:
SOF0, 8-bit samples, Huffman coding, one interleaved scan, restart intervals) step by step in
the order of the standard's decoder:

  1. marker segments (B.2): DQT, SOF0, DHT, DRI, SOS; APPn and COM are skipped;
  2. Huffman tables from BITS and HUFFVAL (Annex C) and the bit-serial DECODE procedure with
     MINCODE / MAXCODE / VALPTR (F.2.2.3); RECEIVE and EXTEND (F.2.2.1, F.2.2.4);
  3. per MCU, per component, per block: the DC difference added to the component's predictor,
     then the AC coefficients with their zero runs, ZRL and EOB (F.2.2.1, F.2.2.2), written to
     natural order through the zig-zag sequence (Figure A.6); at a restart marker the bit
     reader moves to the next byte and the predictors return to 0 (F.2.1.3.1, E.2.4);
  4. dequantisation S = Sq * Q (A.3.4);
  5. the inverse DCT of A.3.3 in exact integer arithmetic: the basis (C_u / 2) cos((2x+1) u pi/16)
     as integers B = round(2^20 * basis), the dequantised coefficient limited to +-16383 (a valid
     stream stays far inside), horizontal sums t = sum_u B[x][u] S[v][u], reduced to
     t' = floor((t + 2^8) / 2^9), vertical sums s = sum_v B[y][v] t'[v][x] (scale 2^31), level
     shift and one rounding floor((s + 128 * 2^31 + 2^30) / 2^31), clamp to 0..255;
  6. components with fewer samples are enlarged by pixel replication (the standard leaves
     upsampling open; replication is the reading taken), planes are cut to the frame size;
  7. YCbCr -> RGB by the JFIF equations on the 8-bit samples with the coefficients as integers
     round(2^16 * c): R = floor((2^16 Y + 91881 Cr' + 2^15) / 2^16), G = floor((2^16 Y -
     22553 Cb' - 46802 Cr' + 2^15) / 2^16), B = floor((2^16 Y + 116130 Cb' + 2^15) / 2^16),
     Cb' = Cb - 128, Cr' = Cr - 128, clamped; a single component goes to all three channels.

Readings where the standard is silent or leaves a choice: the arithmetic of steps 5 and 7, which
the standard only bounds in accuracy (an approximation of the real-valued transform: integers, so
that every decoder following these steps produces the same bytes; `idct_blocks` below is the
real-valued definition in float64 and the pins hold the integer steps to it: a sample differs
from the rounded definition in about one case in a thousand, never by more than one),
replication in step 6, and what is refused (progressive, arithmetic-coded, 12-bit,
four-component, multi-scan frames, DNL).  The decoded bytes are compared bit for bit.

Pins (tests/test_jpeg_oracle_pins.py): hand-built blocks (DC only, one AC coefficient against
the closed form), the inverse transform against scipy's before rounding, an encoder written in
the test (forward DCT from the definition, its own code assignment) whose coefficients must
come back exactly, files written by an image library and its own decode of them, restart
intervals against the same file without them.
"""
from __future__ import annotations

import numpy as np

# zig-zag sequence (Figure A.6): ZIGZAG[k] is the natural-order index (8 * v + u) of the k-th
# coefficient of a block as it is coded
ZIGZAG = [0, 1, 8, 16, 9, 2, 3, 10, 17, 24, 32, 25, 18, 11, 4, 5, 12, 19, 26, 33, 40, 48, 41, 34,
          27, 20, 13, 6, 7, 14, 21, 28, 35, 42, 49, 56, 57, 50, 43, 36, 29, 22, 15, 23, 30, 37,
          44, 51, 58, 59, 52, 45, 38, 31, 39, 46, 53, 60, 61, 54, 47, 55, 62, 63]

# cos(k pi / 16), k = 0..7, correctly rounded to double
_COS = [1.0, 0.9807852804032304, 0.9238795325112867, 0.8314696123025452, 0.7071067811865476,
        0.5555702330196022, 0.3826834323650898, 0.19509032201612828]


def _cos16(k: int) -> float:
    """cos(k pi / 16) for any integer k, from the eight tabulated values by symmetry."""
    k %= 32
    if k > 16:
        k = 32 - k
    return _COS[k] if k <= 8 - 1 else (0.0 if k == 8 else -_COS[16 - k])


def idct_basis() -> np.ndarray:
    """A[x][u] = (C_u / 2) cos((2x + 1) u pi / 16), C_0 = 1/sqrt 2, C_u = 1 otherwise (A.3.3)."""
    a = np.zeros((8, 8), dtype=np.float64)
    for x in range(8):
        for u in range(8):
            a[x, u] = 0.5 * _COS[4] if u == 0 else 0.5 * _cos16((2 * x + 1) * u)
    return a


class Unsupported(ValueError):
    pass


class HuffmanTable:
    """Annex C and F.2.2.3: codes of each length are consecutive integers."""

    def __init__(self, bits: list[int], vals: list[int]):
        if len(bits) != 16 or sum(bits) != len(vals) or len(vals) > 256:
            raise ValueError("bad Huffman table")
        self.bits, self.vals = list(bits), list(vals)
        self.mincode, self.maxcode, self.valptr = [0] * 17, [-1] * 17, [0] * 17
        code, at = 0, 0
        for length in range(1, 17):
            n = bits[length - 1]
            if n:
                self.valptr[length] = at
                self.mincode[length] = code
                code += n
                self.maxcode[length] = code - 1
                at += n
            if code > (1 << length):
                raise ValueError("Huffman code lengths over-subscribed")
            code <<= 1


class Frame:
    def __init__(self):
        self.height = self.width = 0
        self.components: list[dict] = []   # id, h, v, tq, td, ta
        self.qt: dict[int, list[int]] = {}  # natural order
        self.dc: dict[int, HuffmanTable] = {}
        self.ac: dict[int, HuffmanTable] = {}
        self.restart_interval = 0
        self.adobe_transform = 1           # an Adobe segment may say otherwise
        self.scan_start = 0                # index of the first entropy-coded byte

    @property
    def hmax(self):
        return max(c["h"] for c in self.components)

    @property
    def vmax(self):
        return max(c["v"] for c in self.components)

    @property
    def mcus(self) -> tuple[int, int]:
        """(MCU rows, MCU columns) of the frame (A.2.4, A.2.3 for one component)."""
        if len(self.components) == 1:
            return -(-self.height // 8), -(-self.width // 8)
        return -(-self.height // (8 * self.vmax)), -(-self.width // (8 * self.hmax))


def parse(data: bytes) -> Frame:
    """Marker segments up to and including the scan header (B.2)."""
    if len(data) < 4 or data[0] != 0xFF or data[1] != 0xD8:
        raise ValueError("not a JPEG stream (no SOI)")
    f = Frame()
    at, seen_sof = 2, False
    while True:
        if at + 4 > len(data):
            raise ValueError("truncated before the scan")
        if data[at] != 0xFF:
            raise ValueError("marker expected")
        while at < len(data) and data[at + 1] == 0xFF:   # fill bytes
            at += 1
        marker = data[at + 1]
        length = (data[at + 2] << 8) | data[at + 3]
        seg = data[at + 4:at + 2 + length]
        if length < 2 or at + 2 + length > len(data):
            raise ValueError("bad segment length")
        if marker == 0xDB:                                # DQT
            k = 0
            while k < len(seg):
                pq, tq = seg[k] >> 4, seg[k] & 15
                k += 1
                n = 64 * (2 if pq else 1)
                if pq > 1 or tq > 3 or k + n > len(seg):
                    raise ValueError("bad DQT")
                table = [0] * 64
                for z in range(64):
                    q = ((seg[k + 2 * z] << 8) | seg[k + 2 * z + 1]) if pq else seg[k + z]
                    table[ZIGZAG[z]] = q
                f.qt[tq] = table
                k += n
        elif marker == 0xC4:                              # DHT
            k = 0
            while k < len(seg):
                tc, th = seg[k] >> 4, seg[k] & 15
                bits = list(seg[k + 1:k + 17])
                n = sum(bits)
                if tc > 1 or th > 3 or len(bits) != 16 or k + 17 + n > len(seg):
                    raise ValueError("bad DHT")
                table = HuffmanTable(bits, list(seg[k + 17:k + 17 + n]))
                (f.ac if tc else f.dc)[th] = table
                k += 17 + n
        elif marker == 0xC0:                              # SOF0: baseline sequential DCT
            if seen_sof:
                raise Unsupported("more than one frame")
            seen_sof = True
            if seg[0] != 8:
                raise Unsupported("sample precision other than 8 bits")
            f.height, f.width = (seg[1] << 8) | seg[2], (seg[3] << 8) | seg[4]
            nf = seg[5]
            if f.height == 0 or f.width == 0:
                raise Unsupported("frame size left to a DNL segment")
            if nf not in (1, 3) or len(seg) != 6 + 3 * nf:
                raise Unsupported("number of components other than 1 or 3")
            for i in range(nf):
                cid, hv, tq = seg[6 + 3 * i], seg[7 + 3 * i], seg[8 + 3 * i]
                f.components.append({"id": cid, "h": hv >> 4, "v": hv & 15, "tq": tq})
            for c in f.components:
                if c["h"] not in (1, 2) or c["v"] not in (1, 2):
                    raise Unsupported("sampling factors other than 1 and 2")
            if nf == 3:
                c0, c1, c2 = f.components
                if (c1["h"], c1["v"], c2["h"], c2["v"]) != (1, 1, 1, 1):
                    raise Unsupported("chroma sampled more densely than once per MCU")
            else:
                f.components[0]["h"] = f.components[0]["v"] = 1   # A.2.3: one block per MCU
        elif marker in (0xC1, 0xC2, 0xC3, 0xC5, 0xC6, 0xC7, 0xC9, 0xCA, 0xCB, 0xCD, 0xCE, 0xCF):
            raise Unsupported("only baseline sequential DCT frames (SOF0) are decoded")
        elif marker == 0xDD:                              # DRI
            f.restart_interval = (seg[0] << 8) | seg[1]
        elif marker == 0xEE and seg[:5] == b"Adobe" and len(seg) >= 12:
            f.adobe_transform = seg[11]                   # 1: YCbCr, 0: RGB or CMYK as they are
        elif marker == 0xDA:                              # SOS
            if not seen_sof:
                raise ValueError("scan before frame header")
            ns = seg[0]
            if len(f.components) == 3 and f.adobe_transform == 0:
                raise Unsupported("three components that are not YCbCr")
            if ns != len(f.components):
                raise Unsupported("a scan that does not hold every component")
            for j in range(ns):
                cs, tdta = seg[1 + 2 * j], seg[2 + 2 * j]
                if cs != f.components[j]["id"]:
                    raise Unsupported("components of the scan out of frame order")
                f.components[j]["td"], f.components[j]["ta"] = tdta >> 4, tdta & 15
            if (seg[1 + 2 * ns], seg[2 + 2 * ns], seg[3 + 2 * ns]) != (0, 63, 0):
                raise Unsupported("spectral selection or successive approximation")
            f.scan_start = at + 2 + length
            for c in f.components:
                if c["tq"] not in f.qt or c["td"] not in f.dc or c["ta"] not in f.ac:
                    raise ValueError("scan refers to a table that was not defined")
            return f
        elif marker == 0xD9:
            raise ValueError("end of image before any scan")
        # APPn, COM and anything else with a length: skipped
        at += 2 + length


class _Bits:
    """The entropy-coded segment as a bit sequence: a zero byte after 0xFF is stuffing (F.1.2.3);
    any other byte after 0xFF is a marker, and the bits beyond it read as 0."""

    def __init__(self, data: bytes, at: int):
        self.data, self.at = data, at
        self.cur, self.left = 0, 0
        self.marker = None

    def bit(self) -> int:
        if self.left == 0:
            self.cur = 0
            if self.marker is None and self.at < len(self.data):
                b = self.data[self.at]
                if b == 0xFF:
                    nxt = self.data[self.at + 1] if self.at + 1 < len(self.data) else 0xD9
                    if nxt == 0:
                        self.at += 2
                        self.cur = 0xFF
                    else:
                        self.marker = nxt          # stay in front of the marker
                else:
                    self.at += 1
                    self.cur = b
            self.left = 8
        self.left -= 1
        return (self.cur >> self.left) & 1

    def receive(self, n: int) -> int:
        v = 0
        for _ in range(n):
            v = (v << 1) | self.bit()
        return v

    def restart(self, expected: int) -> None:
        """Drop the rest of the byte, pass fill bytes, consume the marker RST_expected (E.2.4)."""
        self.left = 0
        self.marker = None
        while self.at + 1 < len(self.data) and self.data[self.at] == 0xFF \
                and self.data[self.at + 1] == 0xFF:
            self.at += 1
        if self.at + 1 >= len(self.data) or self.data[self.at] != 0xFF \
                or self.data[self.at + 1] != 0xD0 + expected:
            raise ValueError("restart marker missing or out of sequence")
        self.at += 2


def _decode_symbol(bits: _Bits, t: HuffmanTable) -> int:
    code, length = bits.bit(), 1
    while code > t.maxcode[length]:
        length += 1
        if length > 16:
            raise ValueError("code longer than 16 bits")
        code = (code << 1) | bits.bit()
    return t.vals[t.valptr[length] + code - t.mincode[length]]


def _extend(v: int, t: int) -> int:
    return v if t == 0 or v >= (1 << (t - 1)) else v - (1 << t) + 1


def entropy_decode(data: bytes, frame: Frame | None = None) -> list[np.ndarray]:
    """Quantised coefficients of every component, natural order: arrays
    [block rows, block columns, 64] (int32), block counts padded to whole MCUs."""
    f = frame or parse(data)
    mcu_rows, mcu_cols = f.mcus
    planes = [np.zeros((mcu_rows * c["v"], mcu_cols * c["h"], 64), dtype=np.int32)
              for c in f.components]
    bits = _Bits(data, f.scan_start)
    pred = [0] * len(f.components)
    count, rst = 0, 0
    for my in range(mcu_rows):
        for mx in range(mcu_cols):
            if f.restart_interval and count and count % f.restart_interval == 0:
                bits.restart(rst)
                rst = (rst + 1) & 7
                pred = [0] * len(f.components)
            for ci, c in enumerate(f.components):
                dc, ac = f.dc[c["td"]], f.ac[c["ta"]]
                for by in range(c["v"]):
                    for bx in range(c["h"]):
                        block = planes[ci][my * c["v"] + by, mx * c["h"] + bx]
                        t = _decode_symbol(bits, dc)
                        if t > 11:
                            raise ValueError("DC category above 11")
                        pred[ci] += _extend(bits.receive(t), t)
                        block[0] = pred[ci]
                        k = 1
                        while k < 64:
                            rs = _decode_symbol(bits, ac)
                            r, s = rs >> 4, rs & 15
                            if s == 0:
                                if r != 15:
                                    break             # EOB
                                k += 16               # ZRL
                                continue
                            k += r
                            if k > 63:
                                raise ValueError("AC run past the end of the block")
                            block[ZIGZAG[k]] = _extend(bits.receive(s), s)
                            k += 1
            count += 1
    return planes


def idct_blocks(coef: np.ndarray) -> np.ndarray:
    """The real-valued inverse DCT of A.3.3 for blocks [..., 64] of dequantised coefficients
    (natural order 8 v + u) in float64: [..., 8, 8] before the level shift.  The definition the
    integer steps approximate; not used by `decode`."""
    a = idct_basis()
    s = coef.astype(np.float64).reshape(coef.shape[:-1] + (8, 8))   # [.., v, u]
    rows = np.zeros(s.shape, dtype=np.float64)                        # [.., v, x]
    for x in range(8):
        acc = a[x, 0] * s[..., :, 0]
        for u in range(1, 8):
            acc = acc + a[x, u] * s[..., :, u]
        rows[..., :, x] = acc
    out = np.zeros(s.shape, dtype=np.float64)                         # [.., y, x]
    for y in range(8):
        acc = a[y, 0] * rows[..., 0, :]
        for v in range(1, 8):
            acc = acc + a[y, v] * rows[..., v, :]
        out[..., y, :] = acc
    return out


def integer_basis() -> np.ndarray:
    """B[x][u] = round(2^20 * (C_u / 2) cos((2x + 1) u pi / 16))."""
    return np.rint(idct_basis() * float(1 << 20)).astype(np.int64)


def idct_blocks_int(deq: np.ndarray) -> np.ndarray:
    """Step 5's sums for blocks [..., 64] of dequantised coefficients: int64 [..., 8, 8], the
    samples before the level shift times 2^31."""
    b = integer_basis()
    s = np.clip(deq.astype(np.int64), -16383, 16383).reshape(deq.shape[:-1] + (8, 8))  # [.., v, u]
    t = np.einsum("xu,...vu->...vx", b, s)                     # exact: below 2^38
    t = (t + (1 << 8)) >> 9                                    # floor division: below 2^29
    return np.einsum("yv,...vx->...yx", b, t)                  # exact: below 2^52


def samples(coef_q: np.ndarray, qtable: list[int]) -> np.ndarray:
    """One component's sample plane (uint8) from its quantised coefficients: dequantise,
    integer inverse DCT, level shift, one rounding, clamp."""
    q = np.asarray(qtable, dtype=np.int64)
    total = idct_blocks_int(coef_q.astype(np.int64) * q)
    pix = (total + (128 << 31) + (1 << 30)) >> 31
    pix = np.clip(pix, 0, 255).astype(np.uint8)                       # [by, bx, y, x]
    by, bx = pix.shape[0], pix.shape[1]
    return pix.transpose(0, 2, 1, 3).reshape(by * 8, bx * 8)


def ycbcr_to_rgb(y: np.ndarray, cb: np.ndarray, cr: np.ndarray) -> np.ndarray:
    """JFIF: R = Y + 1.402 (Cr - 128), G = Y - 0.344136 (Cb - 128) - 0.714136 (Cr - 128),
    B = Y + 1.772 (Cb - 128), the coefficients as integers round(2^16 c), one rounding
    floor((x + 2^15) / 2^16), clamp."""
    yi = y.astype(np.int64) << 16
    cbi, cri = cb.astype(np.int64) - 128, cr.astype(np.int64) - 128
    r = (yi + 91881 * cri + (1 << 15)) >> 16
    g = (yi - 22553 * cbi - 46802 * cri + (1 << 15)) >> 16
    b = (yi + 116130 * cbi + (1 << 15)) >> 16
    return np.clip(np.stack([r, g, b], axis=-1), 0, 255).astype(np.uint8)


def decode(data: bytes) -> np.ndarray:
    """The decoded image, uint8 [height, width, 3] (RGB)."""
    f = parse(data)
    coef = entropy_decode(data, f)
    planes = []
    for c, cq in zip(f.components, coef):
        p = samples(cq, f.qt[c["tq"]])
        p = np.repeat(np.repeat(p, f.vmax // c["v"], axis=0), f.hmax // c["h"], axis=1)
        planes.append(p[:f.height, :f.width])
    if len(planes) == 1:
        return np.repeat(planes[0][:, :, None], 3, axis=2)
    return ycbcr_to_rgb(*planes)
