"""Pins for the variant oracle (explicit crop origins, resize rounded to uint8).  None of the
expected values below is produced by the function under test: they come from closed forms,
from exact-rational brute force written from the continuous statement, and from sub-windows
of the base oracle's output (a different source file)."""
from __future__ import annotations


import numpy as np
import pytest

import oracle
from oracle import exact_fraction as xf

MEAN = (0.485, 0.456, 0.406)
STD = (0.229, 0.224, 0.225)
M64 = np.asarray(MEAN, dtype=np.float32).astype(np.float64)
S64 = np.asarray(STD, dtype=np.float32).astype(np.float64)


def u8(img, c, s, origin=None):
    co = None if origin is None else [origin]
    return oracle.preprocess_ex([img], c, s, MEAN, STD, oracle.OUT_U8_HWC, crop_origin=co,
                                round_u8=True)[0]


def rand_img(seed, h, w):
    return np.random.default_rng(seed).integers(0, 256, size=(h, w, 3), dtype=np.uint8)


# ---- rounding to uint8 ------------------------------------------------------------------------

def test_identity_gives_the_image_back():
    img = rand_img(1, 16, 16)
    assert np.array_equal(u8(img, 16, 16), img)


def test_pure_crop_at_an_explicit_origin():
    # 12 x 20 with s = 12: R = 12 x 20, scale exactly 1 on both axes
    img = rand_img(2, 12, 20)
    for top, left, c in [(0, 0, 12), (0, 8, 12), (3, 5, 7), (5, 13, 7), (11, 19, 1)]:
        assert np.array_equal(u8(img, c, 12, (top, left)), img[top:top + c, left:left + c])
    # the centre crop is the explicit origin floor((R - c)/2)
    assert np.array_equal(u8(img, 7, 12), img[2:9, 6:13])


def test_constant_image_stays_constant():
    for value in (0, 1, 127, 254, 255):
        img = np.full((9, 13, 3), value, dtype=np.uint8)
        img[..., 1] = 255 - value
        out = u8(img, 11, 17)
        assert np.all(out[..., 0] == value) and np.all(out[..., 1] == 255 - value)


def test_two_times_upscale_of_ramps_with_known_ties():
    """p[y][x] = a + b*x on an n x n image, s = 2n: interior v = a + b*(X/2 - 1/4).
    b = 2: v = a + X - 1/2, a tie, which goes up: a + X.  b = 4: v = a + 2X - 1 exactly.
    b = 1: v = a + X/2 - 1/4: even X -> a + X/2 (down), odd X -> a + (X-1)/2 + 1/4 -> down.
    Ends clamp: X = 0 -> a, X = 2n-1 -> a + b*(n-1)."""
    n, a = 8, 10
    for b, want_interior in ((2, lambda X: a + X), (4, lambda X: a + 2 * X - 1),
                             (1, lambda X: a + X // 2 if X % 2 == 0 else a + (X - 1) // 2)):
        row = (a + b * np.arange(n)).astype(np.uint8)
        img = np.repeat(np.broadcast_to(row[None, :, None], (n, n, 1)), 3, axis=2).copy()
        out = u8(img, 2 * n, 2 * n)
        want = np.array([a] + [want_interior(X) for X in range(1, 2 * n - 1)] + [a + b * (n - 1)])
        assert np.array_equal(out[5, :, 0], want), (b, out[5, :, 0], want)
        # the same ramp along y
        out_t = u8(np.ascontiguousarray(np.transpose(img, (1, 0, 2))), 2 * n, 2 * n)
        assert np.array_equal(out_t[:, 3, 2], want)


@pytest.mark.parametrize("seed,h,w,c,s,origin", [
    (3, 4, 4, 6, 6, None), (4, 5, 7, 4, 6, None), (5, 7, 5, 5, 9, (3, 2)), (6, 3, 11, 3, 3, (0, 7)),
    (7, 6, 6, 2, 13, (11, 0)), (8, 9, 4, 7, 8, (9, 1)), (9, 1, 1, 3, 3, None), (10, 2, 9, 5, 5, (0, 17)),
])
def test_matches_exact_fraction_brute_force(seed, h, w, c, s, origin):
    img = rand_img(seed, h, w)
    top, left = origin if origin is not None else (None, None)
    exact = xf.resized_pixels(img.tolist(), c, s, top, left)
    want = np.array([[[xf.round_half_up(v) for v in px] for px in row] for row in exact])
    assert np.array_equal(u8(img, c, s, origin), want)
    # the unrounded float path at the same origin agrees with the exact value
    out = oracle.preprocess_ex([img], c, s, MEAN, STD, oracle.OUT_F64,
                               crop_origin=None if origin is None else [origin])[0]
    exact_f = np.array([[[float(v) for v in px] for px in row] for row in exact])
    want_f = np.transpose((exact_f / 255.0 - M64) / S64, (2, 0, 1))
    assert np.max(np.abs(out - want_f)) < 1e-12


def test_ties_go_up_in_a_hand_made_case():
    """Two pixels 0 and 1, s = 4 along x: X = 1 samples 1/4*... exactly: sx = (X+1/2)/2 - 1/2
    = 0, 1/4, 3/4, 1 -> values 0, 1/4, 3/4, 1 -> 0, 0, 1, 1.  With pixels 0 and 2: 0, 1/2, 3/2, 2
    -> 0, 1 (tie up), 2 (tie up), 2."""
    def two(v0, v1):
        img = np.zeros((2, 2, 3), dtype=np.uint8)
        img[:, 0], img[:, 1] = v0, v1
        return u8(img, 4, 4)[1, :, 0].tolist()
    assert two(0, 1) == [0, 0, 1, 1]
    assert two(0, 2) == [0, 1, 2, 2]
    assert two(255, 253) == [255, 255, 254, 253]   # 254.5 -> 255, 253.5 -> 254


def test_rounded_pixel_is_within_half_of_the_unrounded_value():
    img = rand_img(11, 37, 53)
    c, s = 24, 29
    q = u8(img, c, s).astype(np.float64)
    base = oracle.preprocess([img], c, s, MEAN, STD)[0]          # base oracle, centre crop
    v = (np.transpose(base, (1, 2, 0)) * S64 + M64) * 255.0
    assert np.max(np.abs(q - v)) <= 0.5 + 1e-9
    clear = np.abs((v + 0.5) - np.round(v + 0.5)) > 1e-6         # away from ties
    assert np.array_equal(q[clear], np.floor(v + 0.5)[clear])


# ---- explicit crop origin ------------------------------------------------------------------------

def test_window_at_an_origin_is_a_sub_window_of_a_larger_centre_crop():
    """The base oracle's centre crop of size C_big starts at floor((R - C_big)/2); a c x c window
    at (top, left) inside it must equal the corresponding slice."""
    img = rand_img(12, 41, 67)
    s, c_big, c = 30, 28, 9
    rh, rw = oracle.resized_size(41, 67, s)                      # 30 x 49
    big = oracle.preprocess([img], c_big, s, MEAN, STD)[0]
    o_top, o_left = (rh - c_big) // 2, (rw - c_big) // 2
    for dt, dl in [(0, 0), (3, 7), (19, 19), (10, 0)]:
        out = oracle.preprocess_ex([img], c, s, MEAN, STD, oracle.OUT_F64,
                                   crop_origin=[(o_top + dt, o_left + dl)])[0]
        assert np.array_equal(out, big[:, dt:dt + c, dl:dl + c])


def test_centre_origin_reproduces_the_base_oracle_bit_for_bit():
    imgs = [rand_img(13, 30, 45), rand_img(14, 50, 31)]
    c, s = 20, 26
    origins = []
    for im in imgs:
        rh, rw = oracle.resized_size(im.shape[0], im.shape[1], s)
        origins.append(((rh - c) // 2, (rw - c) // 2))
    for kind in (oracle.OUT_F64, oracle.OUT_F32, oracle.OUT_F16, oracle.OUT_BF16):
        a = oracle.preprocess(imgs, c, s, MEAN, STD, kind)
        b = oracle.preprocess_ex(imgs, c, s, MEAN, STD, kind, crop_origin=origins)
        d = oracle.preprocess_ex(imgs, c, s, MEAN, STD, kind)
        assert np.array_equal(a.view(np.uint8), b.view(np.uint8))
        assert np.array_equal(a.view(np.uint8), d.view(np.uint8))


def test_origins_outside_the_resized_image_are_refused():
    img = rand_img(15, 10, 10)
    with pytest.raises(ValueError):
        oracle.preprocess_ex([img], 6, 10, MEAN, STD, crop_origin=[(5, 0)])   # 5 + 6 > 10
    with pytest.raises(ValueError):
        oracle.preprocess_ex([img], 6, 10, MEAN, STD, oracle.OUT_U8_HWC)      # uint8 needs rounding


# ---- rounding, then normalising ------------------------------------------------------------------

def test_normalising_the_rounded_pixel():
    """Planar float output after rounding = (q/255 - mean)/std of the uint8 output (pinned
    above), transposed; the float kinds are single roundings of that."""
    imgs = [rand_img(16, 23, 31), rand_img(17, 31, 23)]
    c, s = 12, 15
    origins = [(1, 3), (4, 0)]
    q = oracle.preprocess_ex(imgs, c, s, MEAN, STD, oracle.OUT_U8_HWC, crop_origin=origins,
                             round_u8=True).astype(np.float64)
    want = np.transpose((q / 255.0 - M64) / S64, (0, 3, 1, 2))
    out64 = oracle.preprocess_ex(imgs, c, s, MEAN, STD, oracle.OUT_F64, crop_origin=origins,
                                 round_u8=True)
    assert np.array_equal(out64, want)
    out32 = oracle.preprocess_ex(imgs, c, s, MEAN, STD, oracle.OUT_F32, crop_origin=origins,
                                 round_u8=True)
    assert np.array_equal(out32, want.astype(np.float32))
    out16 = oracle.preprocess_ex(imgs, c, s, MEAN, STD, oracle.OUT_F16, crop_origin=origins,
                                 round_u8=True)
    assert np.array_equal(out16.view(np.uint16), want.astype(np.float16).view(np.uint16))
    bf = oracle.preprocess_ex(imgs, c, s, MEAN, STD, oracle.OUT_BF16, crop_origin=origins,
                              round_u8=True)
    ref = np.fromiter((oracle.round_bf16_bits(v) for v in want.reshape(-1)), dtype=np.uint16)
    assert np.array_equal(bf.reshape(-1), ref)   # the base file's rounding routine, not this one's


def test_batch_position_and_threads_do_not_matter():
    imgs = [rand_img(20 + i, 17 + 3 * i, 29 - 2 * i) for i in range(5)]
    c, s = 10, 14
    origins = [(i % 4, (2 * i) % 5) for i in range(5)]
    whole = oracle.preprocess_ex(imgs, c, s, MEAN, STD, oracle.OUT_U8_HWC, crop_origin=origins,
                                 round_u8=True, nthreads=3)
    for i, im in enumerate(imgs):
        alone = oracle.preprocess_ex([im], c, s, MEAN, STD, oracle.OUT_U8_HWC,
                                     crop_origin=[origins[i]], round_u8=True)[0]
        assert np.array_equal(whole[i], alone)


def test_large_dimensions_need_the_wide_arithmetic():
    """A 1 x 32768 image resized with s = 7: den products pass 2^32; the value is still the
    exact rounded ratio (checked against Fractions on a few pixels)."""
    rng = np.random.default_rng(30)
    img = rng.integers(0, 256, size=(2, 32768, 3), dtype=np.uint8)
    s, c = 7, 7
    rh, rw = oracle.resized_size(2, 32768, s)                    # 7 x 114688
    left = 50001
    out = u8(img, c, s, (0, left))
    for k, j, ch in [(0, 0, 0), (3, 4, 1), (6, 6, 2), (2, 5, 0)]:
        sy = xf.sample_coord_at(2, rh, k)
        sx = xf.sample_coord_at(32768, rw, left + j)
        v = xf.bilinear(img, 2, 32768, sy, sx, ch)
        assert int(out[k, j, ch]) == xf.round_half_up(v)
