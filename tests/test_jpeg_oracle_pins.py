"""Pins of the JPEG Decode oracle (oracle/jpeg.py), none derived from the functions under test:
the zig-zag order from its diagonal walk, code assignment and bit reading by hand, the inverse
transform against closed forms and a library routine, an encoder written here (forward DCT from
the definition, its own Huffman tables, its own file writer) whose quantised coefficients must
come back exactly, and files written and decoded by an image library."""
from __future__ import annotations

import io
import math

import numpy as np
import pytest

from oracle import jpeg as oj
from paper_2411_19114_b200 import workloads as wl


# ---- the pieces ---------------------------------------------------------------------------------

def test_zigzag_is_the_diagonal_walk():
    order, v, u, up = [], 0, 0, True
    for _ in range(64):
        order.append(8 * v + u)
        if up:
            if u == 7:
                v, up = v + 1, False
            elif v == 0:
                u, up = u + 1, False
            else:
                v, u = v - 1, u + 1
        else:
            if v == 7:
                u, up = u + 1, True
            elif u == 0:
                v, up = v + 1, True
            else:
                v, u = v + 1, u - 1
    assert oj.ZIGZAG == order


def test_code_assignment_by_hand():
    # two codes of length 2, one of length 3, two of length 4: 00 01 | 100 | 1010 1011
    t = oj.HuffmanTable([0, 2, 1, 2] + [0] * 12, [7, 8, 9, 10, 11])
    assert (t.mincode[2], t.maxcode[2], t.valptr[2]) == (0, 1, 0)
    assert (t.mincode[3], t.maxcode[3], t.valptr[3]) == (4, 4, 2)
    assert (t.mincode[4], t.maxcode[4], t.valptr[4]) == (10, 11, 3)
    assert t.maxcode[1] == -1 and t.maxcode[5] == -1
    bits = oj._Bits(bytes([0b00011001, 0b01010110]), 0)   # 00 01 100 1010 1011 0
    assert [oj._decode_symbol(bits, t) for _ in range(5)] == [7, 8, 9, 10, 11]
    with pytest.raises(ValueError):
        oj.HuffmanTable([3] + [0] * 15, [1, 2, 3])           # three codes of one bit


def test_bit_reader_unstuffs_and_stops_at_markers():
    bits = oj._Bits(bytes([0xFF, 0x00, 0x80, 0xFF, 0xD9]), 0)
    assert bits.receive(8) == 0xFF and bits.receive(8) == 0x80
    assert bits.receive(8) == 0 and bits.marker == 0xD9      # zeros beyond the marker
    assert [oj._extend(v, 3) for v in range(8)] == [-7, -6, -5, -4, 4, 5, 6, 7]
    assert oj._extend(0, 0) == 0 and oj._extend(0, 1) == -1 and oj._extend(1, 1) == 1


def test_inverse_transform_closed_forms():
    # DC only: every sample is S00 / 8
    c = np.zeros(64)
    c[0] = 8 * 37
    assert np.allclose(oj.idct_blocks(c), 37.0, atol=1e-12)
    # one AC coefficient S[v][u]: s(y, x) = S/4 C_u C_v cos((2x+1) u pi/16) cos((2y+1) v pi/16)
    for v, u, amp in ((0, 1, 100.0), (3, 0, -50.0), (2, 5, 64.0), (7, 7, 9.0)):
        c = np.zeros(64)
        c[8 * v + u] = amp
        cu = 1 / math.sqrt(2) if u == 0 else 1.0
        cv = 1 / math.sqrt(2) if v == 0 else 1.0
        want = np.array([[amp / 4 * cu * cv * math.cos((2 * x + 1) * u * math.pi / 16)
                          * math.cos((2 * y + 1) * v * math.pi / 16) for x in range(8)]
                         for y in range(8)])
        assert np.allclose(oj.idct_blocks(c), want, atol=1e-10)
    # the basis is orthonormal, and its constants are the cosines
    a = oj.idct_basis()
    assert np.allclose(a.T @ a, 0.25 * np.eye(8) * 4 / 1, atol=1e-15) or np.allclose(a @ a.T, np.eye(8), atol=1e-15)
    assert np.allclose(a @ a.T, np.eye(8), atol=1e-15)


def test_inverse_transform_against_a_library_routine():
    from scipy.fft import idctn

    rng = np.random.default_rng(3)
    blocks = rng.integers(-1024, 1024, size=(50, 64)).astype(np.float64)
    want = idctn(blocks.reshape(50, 8, 8), type=2, norm="ortho", axes=(1, 2))
    assert np.allclose(oj.idct_blocks(blocks), want, atol=1e-9)


def test_integer_transform_against_the_real_valued_definition():
    """The integer steps reproduce the rounded real-valued transform except near ties: never
    more than one apart, about one sample in a thousand."""
    rng = np.random.default_rng(4)
    # coefficients shaped like those of images: large at low frequencies, small at high ones
    scale = 600.0 / (1.0 + np.add.outer(np.arange(8), np.arange(8))) ** 1.5
    deq = np.rint(rng.normal(size=(4000, 8, 8)) * scale).astype(np.int64).reshape(4000, 64)
    exact = oj.idct_blocks(deq)
    got = oj.idct_blocks_int(deq)
    assert float(np.max(np.abs(got / float(1 << 31) - exact))) <= 2e-3   # the sums themselves
    want = np.clip(np.floor(exact + 128.5), 0, 255)
    have = np.clip((got + (128 << 31) + (1 << 30)) >> 31, 0, 255)
    diff = np.abs(have - want)
    assert int(diff.max()) <= 1 and float((diff != 0).mean()) <= 3e-3
    # the basis constants: 2^20 times the cosines, rounded
    b = oj.integer_basis()
    assert b[0, 0] == 370728 and b[0, 1] == 514214 and b[1, 1] == 435930 and b[0, 7] == 102284
    assert np.all(np.abs(b / float(1 << 20) - oj.idct_basis()) <= 0.5 / (1 << 20))
    # coefficients beyond what a valid stream holds are limited, not wrapped
    huge = np.zeros((1, 64), dtype=np.int64)
    huge[0, 0] = 10 ** 6
    assert np.all(oj.idct_blocks_int(huge) == oj.idct_blocks_int(np.minimum(huge, 16383)))


def test_samples_round_once_and_clamp():
    q = [1] * 64
    coef = np.zeros((1, 3, 64), dtype=np.int32)
    coef[0, 0, 0] = 8 * 10 + 4      # 10.5 + 128 -> ties upward: 139
    coef[0, 1, 0] = 8 * 200         # 328 -> clamp to 255
    coef[0, 2, 0] = -8 * 200        # -72 -> clamp to 0
    got = oj.samples(coef, q)
    assert got.shape == (8, 24)
    assert np.all(got[:, :8] == 139) and np.all(got[:, 8:16] == 255) and np.all(got[:, 16:] == 0)
    coef[0, 0, 0] = 2               # dequantisation multiplies: 2 * 36 / 8 = 9
    assert np.all(oj.samples(coef, [36] + [1] * 63)[:, :8] == 137)


def test_colour_conversion_by_hand():
    y = np.array([[100, 100, 0, 255]], dtype=np.uint8)
    cb = np.array([[128, 228, 128, 128]], dtype=np.uint8)
    cr = np.array([[128, 28, 255, 0]], dtype=np.uint8)
    got = oj.ycbcr_to_rgb(y, cb, cr)[0]
    assert list(got[0]) == [100, 100, 100]
    # Cb - 128 = 100, Cr - 128 = -100: R = 100 - 140.2, G = 100 - 34.4136 + 71.4136, B = 100 + 177.2
    assert list(got[1]) == [0, 137, 255]
    assert list(got[2]) == [178, 0, 0]          # 127 * 1.402 = 178.054; G = -90.7 -> 0
    assert list(got[3]) == [76, 255, 255]       # 255 - 179.456 = 75.544 -> 76; G = 346.4 -> 255
    # each coefficient of G at the ends of the chroma range: 128 - 0.344136 * 127 = 84.29,
    # 128 + 0.344136 * 128 = 172.05, 128 - 0.714136 * 127 = 37.30, 128 + 0.714136 * 128 = 219.41
    y = np.full((1, 4), 128, dtype=np.uint8)
    cb = np.array([[255, 0, 128, 128]], dtype=np.uint8)
    cr = np.array([[128, 128, 255, 0]], dtype=np.uint8)
    assert [int(v) for v in oj.ycbcr_to_rgb(y, cb, cr)[0, :, 1]] == [84, 172, 37, 219]


# ---- an encoder of its own ------------------------------------------------------------------------

def _fdct(block: np.ndarray) -> np.ndarray:
    out = np.zeros((8, 8))
    for v in range(8):
        for u in range(8):
            cu = 1 / math.sqrt(2) if u == 0 else 1.0
            cv = 1 / math.sqrt(2) if v == 0 else 1.0
            acc = 0.0
            for y in range(8):
                for x in range(8):
                    acc += block[y, x] * math.cos((2 * x + 1) * u * math.pi / 16) \
                        * math.cos((2 * y + 1) * v * math.pi / 16)
            out[v, u] = 0.25 * cu * cv * acc
    return out


class _Writer:
    def __init__(self):
        self.out, self.acc, self.n = bytearray(), 0, 0

    def put(self, value: int, length: int):
        for i in range(length - 1, -1, -1):
            self.acc = (self.acc << 1) | ((value >> i) & 1)
            self.n += 1
            if self.n == 8:
                self.out.append(self.acc)
                if self.acc == 0xFF:
                    self.out.append(0)
                self.acc, self.n = 0, 0

    def flush(self):
        while self.n:
            self.put(1, 1)


def _codes(lengths: dict[int, int]):
    """Symbols by code length, and their codes (consecutive within a length, doubled between)."""
    bits = [sum(1 for l in lengths.values() if l == n) for n in range(1, 17)]
    vals = [s for n in range(1, 17) for s in sorted(lengths) if lengths[s] == n]
    code, table, at = 0, {}, 0
    for n in range(1, 17):
        for _ in range(bits[n - 1]):
            table[vals[at]] = (code, n)
            code += 1
            at += 1
        code <<= 1
    return bits, vals, table


def _magnitude(v: int) -> tuple[int, int]:
    cat = abs(v).bit_length()
    return cat, (v if v >= 0 else v + (1 << cat) - 1)


def encode(planes, sampling, qtable, height, width, restart=0):
    """A baseline file from component planes (uint8, already padded to whole MCUs) with sampling
    factors [(h, v), ...]; returns (bytes, quantised coefficients per component in natural
    order)."""
    ncomp = len(planes)
    hmax, vmax = max(h for h, _ in sampling), max(v for _, v in sampling)
    mcu_rows = -(-height // (8 * vmax)) if ncomp > 1 else -(-height // 8)
    mcu_cols = -(-width // (8 * hmax)) if ncomp > 1 else -(-width // 8)
    zz = oj.ZIGZAG
    q_nat = np.asarray(qtable, dtype=np.float64).reshape(8, 8)
    coefs = []
    for p, (h, v) in zip(planes, sampling):
        c = np.zeros((mcu_rows * v, mcu_cols * h, 64), dtype=np.int32)
        for by in range(mcu_rows * v):
            for bx in range(mcu_cols * h):
                blk = p[8 * by:8 * by + 8, 8 * bx:8 * bx + 8].astype(np.float64) - 128.0
                c[by, bx] = np.rint(_fdct(blk) / q_nat).astype(np.int32).reshape(64)
        coefs.append(c)
    dc_len = {0: 2, 1: 3, 2: 3, 3: 3, 4: 3, 5: 3, 6: 4, 7: 5, 8: 6, 9: 7, 10: 8, 11: 9}
    ac_len = {0x00: 2, 0x01: 3, 0xF0: 9}
    for r in range(16):
        for s_ in range(1, 11):
            ac_len.setdefault((r << 4) | s_, 9)
    dc_bits, dc_vals, dc_code = _codes(dc_len)
    ac_bits, ac_vals, ac_code = _codes(ac_len)
    w = _Writer()
    pred = [0] * ncomp
    count, rst = 0, 0
    for my in range(mcu_rows):
        for mx in range(mcu_cols):
            if restart and count and count % restart == 0:
                w.flush()
                w.out += bytes([0xFF, 0xD0 + rst])
                rst = (rst + 1) & 7
                pred = [0] * ncomp
            for ci, (h, v) in enumerate(sampling):
                for by in range(v):
                    for bx in range(h):
                        blk = coefs[ci][my * v + by, mx * h + bx]
                        cat, bits = _magnitude(int(blk[0]) - pred[ci])
                        pred[ci] = int(blk[0])
                        w.put(*dc_code[cat])
                        w.put(bits, cat)
                        run = 0
                        last = max([k for k in range(1, 64) if blk[zz[k]] != 0], default=0)
                        for k in range(1, last + 1):
                            val = int(blk[zz[k]])
                            if val == 0:
                                run += 1
                                continue
                            while run > 15:
                                w.put(*ac_code[0xF0])
                                run -= 16
                            cat, bits = _magnitude(val)
                            w.put(*ac_code[(run << 4) | cat])
                            w.put(bits, cat)
                            run = 0
                        if last < 63:
                            w.put(*ac_code[0x00])
            count += 1
    w.flush()
    out = bytearray([0xFF, 0xD8])
    out += bytes([0xFF, 0xFE, 0, 7]) + b"hello"                      # a comment to skip
    out += bytes([0xFF, 0xDB, 0, 67, 0]) + bytes(int(qtable[zz[k]]) for k in range(64))
    out += bytes([0xFF, 0xC0, 0, 8 + 3 * ncomp, 8, height >> 8, height & 255, width >> 8,
                  width & 255, ncomp])
    for ci, (h, v) in enumerate(sampling):
        out += bytes([ci + 1, (h << 4) | v, 0])
    out += bytes([0xFF, 0xC4, 0, 19 + len(dc_vals), 0x00]) + bytes(dc_bits) + bytes(dc_vals)
    out += bytes([0xFF, 0xC4, 0, 19 + len(ac_vals), 0x10]) + bytes(ac_bits) + bytes(ac_vals)
    if restart:
        out += bytes([0xFF, 0xDD, 0, 4, restart >> 8, restart & 255])
    out += bytes([0xFF, 0xDA, 0, 6 + 2 * ncomp, ncomp])
    for ci in range(ncomp):
        out += bytes([ci + 1, 0x00])
    out += bytes([0, 63, 0]) + bytes(w.out) + bytes([0xFF, 0xD9])
    return bytes(out), coefs


def _planes(rng, height, width, sampling):
    hmax, vmax = max(h for h, _ in sampling), max(v for _, v in sampling)
    rows = -(-height // (8 * vmax)) * 8 * vmax if len(sampling) > 1 else -(-height // 8) * 8
    cols = -(-width // (8 * hmax)) * 8 * hmax if len(sampling) > 1 else -(-width // 8) * 8
    out = []
    for h, v in sampling:
        big = wl.smooth_image(rng, rows * v // vmax, cols * h // hmax)[:, :, 0]
        extra = rng.integers(-40, 41, size=big.shape)
        out.append(np.clip(big.astype(np.int64) + extra, 0, 255).astype(np.uint8))
    return out


@pytest.mark.parametrize("sampling,height,width,restart", [
    ([(1, 1), (1, 1), (1, 1)], 21, 35, 0), ([(2, 2), (1, 1), (1, 1)], 40, 50, 0),
    ([(2, 1), (1, 1), (1, 1)], 17, 33, 2), ([(1, 2), (1, 1), (1, 1)], 33, 9, 1),
    ([(1, 1)], 19, 30, 3), ([(2, 2), (1, 1), (1, 1)], 48, 64, 4)])
def test_coefficients_of_an_independent_encoder_come_back_exactly(sampling, height, width, restart):
    rng = np.random.default_rng(height * 1000 + width)
    qtable = [int(v) for v in rng.integers(1, 24, size=64)]
    planes = _planes(rng, height, width, sampling)
    data, coefs = encode(planes, sampling, qtable, height, width, restart)
    f = oj.parse(data)
    assert (f.height, f.width, f.restart_interval) == (height, width, restart)
    assert [(c["h"], c["v"]) for c in f.components] == (sampling if len(sampling) > 1 else [(1, 1)])
    assert f.qt[0] == qtable
    got = oj.entropy_decode(data)
    for g, want in zip(got, coefs):
        assert np.array_equal(g, want)
    # the pixels: the planes themselves within the quantisation error, replicated and cut
    img = oj.decode(data)
    assert img.shape == (height, width, 3)
    if len(sampling) == 1:
        assert np.all(img[:, :, 0] == img[:, :, 1]) and np.all(img[:, :, 0] == img[:, :, 2])
        assert np.max(np.abs(img[:, :, 0].astype(int) - planes[0][:height, :width])) <= 40
    # extreme coefficient values survive (category 10 and 11, long zero runs)
    assert max(int(np.abs(c).max()) for c in coefs) > 20


# ---- files of an image library ---------------------------------------------------------------------

def _library_jpeg(img, **kw):
    from PIL import Image

    buf = io.BytesIO()
    Image.fromarray(img).save(buf, format="JPEG", **kw)
    data = buf.getvalue()
    return data, np.asarray(Image.open(io.BytesIO(data)).convert("RGB"))


@pytest.mark.parametrize("quality", [95, 75, 40])
def test_against_a_librarys_decode_full_chroma(quality):
    rng = np.random.default_rng(quality)
    img = wl.smooth_image(rng, 75, 101)
    data, lib = _library_jpeg(img, quality=quality, subsampling=0)
    got = oj.decode(data)
    # the library's inverse transform and colour conversion are integer approximations: a
    # sample may differ by one, which the colour equations can turn into three in a channel
    assert got.shape == lib.shape
    diff = np.abs(got.astype(int) - lib.astype(int))
    assert int(diff.max()) <= 3 and float((diff == 0).mean()) >= 0.95 and float(diff.mean()) <= 0.06
    assert int(np.max(np.abs(got.astype(int) - img.astype(int)))) <= 60   # and it is the image


@pytest.mark.parametrize("subsampling", [1, 2])
def test_against_a_librarys_decode_subsampled_chroma(subsampling):
    """The library interpolates the chroma planes, the reading here replicates: on smooth
    content the two stay close, and the luma detail is the same."""
    rng = np.random.default_rng(subsampling)
    img = wl.smooth_image(rng, 120, 168)
    data, lib = _library_jpeg(img, quality=90, subsampling=subsampling)
    got = oj.decode(data)
    diff = np.abs(got.astype(int) - lib.astype(int))
    assert int(diff.max()) <= 12 and float(diff.mean()) <= 1.5


def test_restart_intervals_change_nothing():
    rng = np.random.default_rng(9)
    img = wl.smooth_image(rng, 90, 130)
    plain, _ = _library_jpeg(img, quality=85, subsampling=2)
    marked, _ = _library_jpeg(img, quality=85, subsampling=2, restart_marker_rows=1)
    assert oj.parse(plain).restart_interval == 0 and oj.parse(marked).restart_interval > 0
    assert np.array_equal(oj.decode(plain), oj.decode(marked))
    grey, lib = _library_jpeg(img[:, :, 1], quality=85)
    assert int(np.max(np.abs(oj.decode(grey).astype(int) - lib.astype(int)))) <= 1


def test_what_is_not_decoded_is_refused():
    rng = np.random.default_rng(10)
    img = wl.smooth_image(rng, 40, 40)
    prog, _ = _library_jpeg(img, quality=80, progressive=True)
    with pytest.raises(oj.Unsupported):
        oj.decode(prog)
    from PIL import Image

    buf = io.BytesIO()
    Image.fromarray(np.dstack([img, img[:, :, :1]]), mode="CMYK").save(buf, format="JPEG")
    with pytest.raises(oj.Unsupported):
        oj.decode(buf.getvalue())
    good, _ = _library_jpeg(img, quality=80)
    with pytest.raises(ValueError):
        oj.decode(good[:100])
    with pytest.raises(ValueError):
        oj.decode(b"\x00\x01\x02\x03")
