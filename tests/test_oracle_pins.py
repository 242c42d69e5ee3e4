"""Pins for the CPU oracle: closed forms, invariants, exact brute force, hand-worked
pixels and a library special case.  None of the expected values below is produced by
the function under test."""
from __future__ import annotations

import struct
from fractions import Fraction
from pathlib import Path

import numpy as np
import pytest

import oracle
from oracle import exact_fraction as xf

MEAN = (0.485, 0.456, 0.406)
STD = (0.229, 0.224, 0.225)
M64 = np.asarray(MEAN, dtype=np.float32).astype(np.float64)
S64 = np.asarray(STD, dtype=np.float32).astype(np.float64)
GOLDEN = Path(__file__).parent / "golden"


def normalise(v: np.ndarray) -> np.ndarray:
    """(v/255 - mean)/std on an HWC array of pixel-unit values -> CHW, in float64."""
    return np.transpose((v / 255.0 - M64) / S64, (2, 0, 1))


def to_pixels(out: np.ndarray) -> np.ndarray:
    """Invert the normalisation of a CHW result back to pixel units (HWC)."""
    return (np.transpose(out, (1, 2, 0)) * S64 + M64) * 255.0


def run1(img, c, s, mean=MEAN, std=STD):
    return oracle.preprocess([img], c, s, mean, std)[0]


# ---- resized size and crop origin ---------------------------------------------------------

def test_resized_size_floor_rule():
    assert oracle.resized_size(240, 320, 256) == (256, 341)      # 256*320/240 = 341.33
    assert oracle.resized_size(375, 500, 256) == (256, 341)
    assert oracle.resized_size(1080, 1920, 256) == (256, 455)    # 455.11
    assert oracle.resized_size(500, 375, 256) == (341, 256)      # portrait
    assert oracle.resized_size(300, 300, 256) == (256, 256)
    assert oracle.resized_size(3, 5, 7) == (7, 11)               # 35/3 = 11.67 -> 11, not 12


def test_axis_invariants():
    for n_in, r, c in [(240, 256, 224), (320, 341, 224), (1920, 455, 224), (7, 7, 7), (5, 40, 33),
                       (1, 9, 9), (32768, 256, 224)]:
        prev = -1.0
        for j in range(c):
            i0, i1, lam = oracle.axis(n_in, r, c, j)
            assert 0 <= i0 <= i1 <= n_in - 1 and i1 - i0 <= 1
            assert 0.0 <= lam < 1.0
            pos = i0 + lam
            assert pos >= prev  # monotone sampling positions
            prev = pos
            # position equals the clamped half-pixel formula, evaluated exactly
            want = xf.sample_coord(n_in, r, c, j)
            assert abs(Fraction(pos) - want) < Fraction(1, 10**9)


# ---- P1 identity ----------------------------------------------------------------------------

def test_identity_when_sizes_match():
    rng = np.random.default_rng(11)
    img = rng.integers(0, 256, size=(24, 24, 3), dtype=np.uint8)
    out = run1(img, 24, 24)
    want = normalise(img.astype(np.float64))
    assert out.shape == (3, 24, 24)
    assert np.array_equal(out, want)  # lambda == 0 everywhere: exact


# ---- P2 pure crop -----------------------------------------------------------------------------

@pytest.mark.parametrize("h,w,s,c", [(16, 24, 16, 10), (24, 16, 16, 10), (16, 24, 16, 11),
                                     (256, 341 * 3, 256, 224)])
def test_pure_crop_when_scale_is_one(h, w, s, c):
    rng = np.random.default_rng(12)
    img = rng.integers(0, 256, size=(h, w, 3), dtype=np.uint8)
    rh, rw = (s, s * w // h) if h <= w else (s * h // w, s)
    assert (rh, rw) == (h, w)
    top, left = (rh - c) // 2, (rw - c) // 2
    want = normalise(img[top:top + c, left:left + c].astype(np.float64))
    assert np.array_equal(run1(img, c, s), want)


# ---- P3 constant images -----------------------------------------------------------------------

@pytest.mark.parametrize("h,w", [(5, 9), (31, 17), (240, 320)])
def test_constant_image_is_exact(h, w):
    for value in (0, 1, 127, 254, 255):
        img = np.full((h, w, 3), value, dtype=np.uint8)
        img[..., 1] = 255 - value
        out = run1(img, 14, 19)
        for ch, pv in enumerate((value, 255 - value, value)):
            want = (pv / 255.0 - M64[ch]) / S64[ch]
            assert np.all(out[ch] == want)


# ---- P4 2x upscale of a ramp ------------------------------------------------------------------

@pytest.mark.parametrize("axis", [0, 1])
def test_two_times_upscale_of_ramp(axis):
    n, a, b = 12, 7, 20
    ramp = a + b * np.arange(n)
    img = np.zeros((n, n, 3), dtype=np.uint8)
    img[:] = ramp[:, None, None] if axis == 0 else ramp[None, :, None]
    out = to_pixels(run1(img, 2 * n, 2 * n))
    X = np.arange(2 * n, dtype=np.float64)
    want = a + b * (X / 2 - 0.25)
    want[0], want[-1] = a, a + b * (n - 1)
    line = out[:, 3, 0] if axis == 0 else out[5, :, 2]
    assert np.allclose(line, want, rtol=0, atol=1e-10)
    # weights alternate 3/4, 1/4 in the interior
    lams = [oracle.axis(n, 2 * n, 2 * n, j)[2] for j in range(1, 2 * n - 1)]
    assert lams == [0.25, 0.75] * (n - 1)


# ---- P5 affine reproduction -------------------------------------------------------------------

@pytest.mark.parametrize("h,w,s,c", [(13, 17, 20, 16), (17, 13, 20, 16), (60, 45, 21, 21),
                                     (40, 100, 16, 9)])
def test_affine_image_is_reproduced(h, w, s, c):
    a, bx, by = 3.0, 1.0, 2.0
    yy, xx = np.mgrid[0:h, 0:w]
    plane = a + bx * xx + by * yy
    assert plane.max() <= 255
    img = np.repeat(plane[..., None], 3, axis=2).astype(np.uint8)
    out = to_pixels(run1(img, c, s))
    rh, rw = (s, s * w // h) if h <= w else (s * h // w, s)
    top, left = (rh - c) // 2, (rw - c) // 2
    sx = np.clip((np.arange(c) + left + 0.5) * w / rw - 0.5, 0, w - 1)
    sy = np.clip((np.arange(c) + top + 0.5) * h / rh - 0.5, 0, h - 1)
    want = a + bx * sx[None, :] + by * sy[:, None]
    for ch in range(3):
        assert np.allclose(out[..., ch], want, rtol=0, atol=1e-9)


# ---- P6 exact-rational brute force and hand-worked pixels ---------------------------------------

@pytest.mark.parametrize("seed", range(12))
def test_matches_exact_fraction_brute_force(seed):
    rng = np.random.default_rng(100 + seed)
    h, w = (int(v) for v in rng.integers(1, 13, size=2))
    s = int(rng.integers(1, 17))
    rh, rw = xf.resized_size(h, w, s)
    c = int(rng.integers(1, min(rh, rw, s) + 1))
    img = rng.integers(0, 256, size=(h, w, 3), dtype=np.uint8)
    mean = rng.uniform(0.2, 0.7, size=3).astype(np.float32)
    std = rng.uniform(0.1, 0.5, size=3).astype(np.float32)
    got = run1(img, c, s, mean, std)
    want = xf.preprocess(img.tolist(), c, s, mean, std)
    for ch in range(3):
        for k in range(c):
            for j in range(c):
                assert abs(Fraction(got[ch, k, j]) - want[ch][k][j]) < Fraction(1, 10**12)


def test_matches_exact_fraction_on_hypothesis_cases():
    hyp = pytest.importorskip("hypothesis")
    st = hyp.strategies

    @hyp.settings(max_examples=60, deadline=None, derandomize=True)
    @hyp.given(h=st.integers(1, 9), w=st.integers(1, 9), s=st.integers(1, 12), seed=st.integers(0, 10**6),
               frac=st.floats(0.0, 1.0))
    def check(h, w, s, seed, frac):
        rh, rw = xf.resized_size(h, w, s)
        c = max(1, min(rh, rw, s, int(round(frac * s)) or 1))
        img = np.random.default_rng(seed).integers(0, 256, size=(h, w, 3), dtype=np.uint8)
        got = run1(img, c, s)
        # the constants as the float32 values the interface carries
        want = xf.preprocess(img.tolist(), c, s, np.float32(MEAN), np.float32(STD))
        for ch in range(3):
            for k in range(c):
                for j in range(c):
                    assert abs(Fraction(got[ch, k, j]) - want[ch][k][j]) < Fraction(1, 10**12)

    check()


def _read_hand_cases():
    planes = {"R": {}, "G": {}, "B": {}}
    cases, expects = {}, []
    for raw in (GOLDEN / "hand_4x4.txt").read_text().splitlines():
        t = raw.split("#")[0].split()
        if not t:
            continue
        if t[0] == "image":
            planes[t[1]][int(t[2])] = [int(v) for v in t[3:]]
        elif t[0] == "case":
            cases[t[1]] = dict(rows=(int(t[3]), int(t[4])), cols=(int(t[6]), int(t[7])),
                               s=int(t[9]), c=int(t[11]))
        elif t[0] == "expect":
            expects.append((t[1], "RGB".index(t[2]), int(t[3]), int(t[4]), Fraction(t[5])))
    img = np.zeros((4, 4, 3), dtype=np.uint8)
    for ch, name in enumerate("RGB"):
        for y in range(4):
            img[y, :, ch] = planes[name][y]
    return img, cases, expects


def test_hand_worked_pixels():
    img, cases, expects = _read_hand_cases()
    assert len(expects) >= 30
    outs = {}
    for name, cs in cases.items():
        sub = img[cs["rows"][0]:cs["rows"][1], cs["cols"][0]:cs["cols"][1]]
        outs[name] = to_pixels(run1(sub, cs["c"], cs["s"]))
    for name, ch, k, j, want in expects:
        assert abs(outs[name][k, j, ch] - float(want)) < 1e-10, (name, ch, k, j)


# ---- P7 flip symmetry and the floor rule of the crop origin -------------------------------------

def test_flip_symmetry_even_and_odd_margin():
    rng = np.random.default_rng(13)
    # (R_w - C) even: 30x40 -> R = 24x32, C = 20 -> margin 12
    img = rng.integers(0, 256, size=(30, 40, 3), dtype=np.uint8)
    a = run1(img, 20, 24)
    b = run1(img[:, ::-1].copy(), 20, 24)
    assert np.allclose(b, a[:, :, ::-1], rtol=0, atol=1e-12)
    # (R_w - C) odd: C = 21 -> margin 11, origin 5: window is biased one pixel to the left,
    # so the flipped input's column j is the original's column C - j (j >= 1).
    a = run1(img, 21, 24)
    b = run1(img[:, ::-1].copy(), 21, 24)
    assert np.allclose(b[:, :, 1:], a[:, :, :0:-1], rtol=0, atol=1e-12)
    assert not np.allclose(b, a[:, :, ::-1], rtol=0, atol=1e-3)


# ---- P8 range / convexity -----------------------------------------------------------------------

def test_values_stay_within_their_four_taps():
    rng = np.random.default_rng(14)
    h, w, s, c = 37, 23, 19, 15
    img = rng.integers(0, 256, size=(h, w, 3), dtype=np.uint8)
    out = to_pixels(run1(img, c, s))
    rh, rw = xf.resized_size(h, w, s)
    for k in range(c):
        sy = xf.sample_coord(h, rh, c, k)
        y0 = int(sy)
        y1 = min(y0 + 1, h - 1)
        for j in range(c):
            sx = xf.sample_coord(w, rw, c, j)
            x0 = int(sx)
            x1 = min(x0 + 1, w - 1)
            block = img[[y0, y0, y1, y1], [x0, x1, x0, x1]].astype(np.float64)
            assert np.all(out[k, j] >= block.min(axis=0) - 1e-9)
            assert np.all(out[k, j] <= block.max(axis=0) + 1e-9)


# ---- P9 independence of batch position, channel permutation ---------------------------------------

def test_batch_position_and_channel_permutation():
    rng = np.random.default_rng(15)
    a = rng.integers(0, 256, size=(19, 31, 3), dtype=np.uint8)
    b = rng.integers(0, 256, size=(40, 17, 3), dtype=np.uint8)
    c = rng.integers(0, 256, size=(16, 16, 3), dtype=np.uint8)
    alone = oracle.preprocess([a], 12, 16, MEAN, STD)[0]
    for batch, idx in (([a, b, c], 0), ([b, a, c], 1), ([c, b, a], 2)):
        for threads in (1, 3):
            got = oracle.preprocess(batch, 12, 16, MEAN, STD, nthreads=threads)[idx]
            assert np.array_equal(got, alone)
    perm = [2, 0, 1]
    got = oracle.preprocess([a[..., perm].copy()], 12, 16, [MEAN[p] for p in perm],
                            [STD[p] for p in perm])[0]
    assert np.array_equal(got, alone[perm])


# ---- P10 library special case: torch's bilinear interpolate in float64 ------------------------------

@pytest.mark.parametrize("h,w", [(240, 320), (375, 500), (333, 471), (471, 333), (250, 250),
                                 (1080, 1920), (100, 90)])
def test_against_torch_interpolate_float64(h, w):
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(16)
    s, c = 256, 224
    img = rng.integers(0, 256, size=(h, w, 3), dtype=np.uint8)
    rh, rw = (s, s * w // h) if h <= w else (s * h // w, s)
    x = torch.from_numpy(img.astype(np.float64)).permute(2, 0, 1)[None]
    y = torch.nn.functional.interpolate(x, size=(rh, rw), mode="bilinear", align_corners=False,
                                        antialias=False)[0].numpy()
    top, left = (rh - c) // 2, (rw - c) // 2
    want = (y[:, top:top + c, left:left + c] / 255.0 - M64[:, None, None]) / S64[:, None, None]
    got = run1(img, c, s)
    assert np.max(np.abs(got - want)) < 1e-9


# ---- P11 packing -------------------------------------------------------------------------------------

def test_pack_layout():
    rng = np.random.default_rng(17)
    sizes = [(1, 1), (5, 7), (128, 1), (3, 43), (16, 8), (2, 64)]
    imgs = [rng.integers(0, 256, size=(h, w, 3), dtype=np.uint8) for h, w in sizes]
    packed, offsets, hh, ww = oracle.pack(imgs)
    at = 0
    covered = np.zeros(len(packed), dtype=bool)
    for i, (h, w) in enumerate(sizes):
        assert offsets[i] == at and at % 128 == 0
        assert (hh[i], ww[i]) == (h, w)
        nbytes = 3 * h * w
        assert np.array_equal(packed[at:at + nbytes], imgs[i].reshape(-1))
        # element (y, x, ch) sits at offset + 3*(y*w + x) + ch
        y, x, ch = h - 1, w // 2, 1
        assert packed[at + 3 * (y * w + x) + ch] == imgs[i][y, x, ch]
        covered[at:at + nbytes] = True
        at = -(-(at + nbytes) // 128) * 128
    assert len(packed) == at
    assert np.all(packed[~covered] == 0)


# ---- rounding to binary16 -----------------------------------------------------------------------------

def _half_bits_struct(x: float) -> int:
    try:
        return struct.unpack("<H", struct.pack("<e", x))[0]
    except OverflowError:
        return 0xFC00 if x < 0 else 0x7C00


def test_round_to_binary16_matches_two_other_implementations():
    rng = np.random.default_rng(18)
    vals = list(rng.uniform(-3, 3, size=2000)) + list(rng.uniform(-1e-4, 1e-4, size=2000))
    vals += list(rng.uniform(-7e4, 7e4, size=500)) + list(rng.normal(size=500) * 1e-7)
    # exact halves between neighbours, subnormal boundaries, overflow threshold, zeros
    for bits in (0x0001, 0x03FF, 0x0400, 0x3BFF, 0x3C00, 0x4200, 0x7BFE, 0x7BFF):
        lo = float(np.uint16(bits).view(np.float16))
        hi = float(np.uint16(bits + 1).view(np.float16)) if bits < 0x7BFF else 65536.0
        vals += [lo, (lo + hi) / 2, np.nextafter((lo + hi) / 2, 0), np.nextafter((lo + hi) / 2, 1e9)]
    vals += [0.0, -0.0, 2.0 ** -25, np.nextafter(2.0 ** -25, 1), -(2.0 ** -25), 65519.99, 65520.0,
             1e6, -1e6]
    for v in vals:
        v = float(v)
        got = oracle.round_f16_bits(v)
        with np.errstate(over="ignore"):
            assert got == int(np.float64(v).astype(np.float16).view(np.uint16)), v
        assert got == _half_bits_struct(v), v


def test_round_to_bfloat16():
    torch = pytest.importorskip("torch")
    # hand cases: 1 + 2^-8 is halfway between 1 and 1 + 2^-7 -> even (1.0); 1 + 3*2^-8 -> 1 + 2^-6
    assert oracle.round_bf16_bits(1.0) == 0x3F80
    assert oracle.round_bf16_bits(1.0 + 2.0 ** -8) == 0x3F80
    assert oracle.round_bf16_bits(np.nextafter(1.0 + 2.0 ** -8, 2.0)) == 0x3F81
    assert oracle.round_bf16_bits(1.0 + 3 * 2.0 ** -8) == 0x3F82
    assert oracle.round_bf16_bits(-2.5) == 0xC020
    assert oracle.round_bf16_bits(0.0) == 0 and oracle.round_bf16_bits(-0.0) == 0x8000
    assert oracle.round_bf16_bits(3.5e38) == 0x7F80           # beyond the largest finite value
    assert oracle.round_bf16_bits(2.0 ** -133) == 0x0001       # smallest subnormal
    assert oracle.round_bf16_bits(2.0 ** -134) == 0x0000       # half of it: tie to even (zero)
    # a library's conversion on values that are exact in float32 (so no second rounding)
    rng = np.random.default_rng(20)
    vals = np.concatenate([rng.uniform(-3, 3, 3000), rng.normal(size=1000) * 1e-3,
                           rng.uniform(-1e30, 1e30, 200)]).astype(np.float32)
    want = torch.from_numpy(vals).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = np.array([oracle.round_bf16_bits(float(v)) for v in vals], dtype=np.uint16)
    assert np.array_equal(got, want)


def test_output_kinds_are_single_roundings():
    rng = np.random.default_rng(19)
    imgs = [rng.integers(0, 256, size=(20, 27, 3), dtype=np.uint8) for _ in range(3)]
    f64 = oracle.preprocess(imgs, 12, 14, MEAN, STD, oracle.OUT_F64)
    f32 = oracle.preprocess(imgs, 12, 14, MEAN, STD, oracle.OUT_F32, nthreads=2)
    f16 = oracle.preprocess(imgs, 12, 14, MEAN, STD, oracle.OUT_F16, nthreads=3)
    assert f32.dtype == np.float32 and np.array_equal(f32, f64.astype(np.float32))
    assert f16.dtype == np.float16 and np.array_equal(f16, f64.astype(np.float16))
    bf = oracle.preprocess(imgs, 12, 14, MEAN, STD, oracle.OUT_BF16)
    assert bf.dtype == np.uint16
    assert all(int(b) == oracle.round_bf16_bits(float(v)) for b, v in zip(bf.ravel(), f64.ravel()))


def test_rejects_bad_arguments():
    img = np.zeros((8, 8, 3), dtype=np.uint8)
    with pytest.raises(ValueError):
        oracle.preprocess([img], 9, 8, MEAN, STD)           # crop larger than resize
    with pytest.raises(ValueError):
        oracle.preprocess([img], 4, 8, MEAN, (0.2, 0.0, 0.2))  # zero std
