"""Pins for the antialiased-Resize oracle.  No expected value below is produced by the module
under test: they are closed forms worked by hand, an exact-rational restatement of the
continuous definition, a library routine (torch's antialiased interpolation on the CPU, in
float64), and the plain transform's oracle (a C file) where no axis is reduced."""
from __future__ import annotations

from fractions import Fraction

import numpy as np
import pytest

import oracle
from oracle import antialias as aa

MEAN = (0.485, 0.456, 0.406)
STD = (0.229, 0.224, 0.225)
M64 = np.asarray(MEAN, dtype=np.float32).astype(np.float64)
S64 = np.asarray(STD, dtype=np.float32).astype(np.float64)


def rand_img(seed, h, w):
    return np.random.default_rng(seed).integers(0, 256, size=(h, w, 3), dtype=np.uint8)


# ---- the weights ----------------------------------------------------------------------------------

def test_halving_has_the_one_three_three_one_kernel():
    """n_in = 16 -> R = 8: sigma = 2, c = 2X + 1; pixel centres at distance 1/2, 3/2 on each side
    weigh 3/4 and 1/4; normalised by their sum 2."""
    w = aa.axis_weights(16, 8, 0, 8)
    assert w.shape == (8, 16)
    for x in range(1, 7):
        want = np.zeros(16)
        want[2 * x - 1:2 * x + 3] = [1 / 8, 3 / 8, 3 / 8, 1 / 8]
        assert np.allclose(w[x], want, atol=1e-15)
    # at the border the missing pixel's weight is shared out: (3/4, 3/4, 1/4) / (7/4)
    want = np.zeros(16)
    want[:3] = [3 / 7, 3 / 7, 1 / 7]
    assert np.allclose(w[0], want, atol=1e-15)
    assert np.allclose(w[7], want[::-1], atol=1e-15)


def test_reduction_by_three():
    """sigma = 3, c = 3X + 3/2 = 13.5 for X = 4, the centre of pixel 13: distances 0, 1, 2 ->
    1, 2/3, 1/3; sum 3."""
    w = aa.axis_weights(30, 10, 4, 1)[0]
    want = np.zeros(30)
    want[11:16] = np.array([1, 2, 3, 2, 1]) / 9
    assert np.allclose(w, want, atol=1e-15)


def test_no_reduction_gives_the_two_tap_weights():
    """n_in = 4 -> R = 8: sigma = 1, c = X/2 + 1/4: X = 3 -> c = 7/4 -> pixels 0 (dist 5/4: none),
    1 (centre 3/2, dist 1/4 -> 3/4), 2 (centre 5/2, dist 3/4 -> 1/4); X = 0 -> c = 1/4 -> pixel 0
    alone (dist 1/4 -> 3/4, normalised to 1): the clamped border."""
    w = aa.axis_weights(4, 8, 0, 8)
    assert np.allclose(w[3], [0, 0.75, 0.25, 0], atol=1e-15)
    assert np.allclose(w[0], [1, 0, 0, 0], atol=1e-15)
    assert np.allclose(w[7], [0, 0, 0, 1], atol=1e-15)


@pytest.mark.parametrize("n_in,r", [(7, 3), (10, 4), (33, 5), (9, 9), (5, 8), (1, 3), (100, 7)])
def test_weights_against_exact_fractions(n_in, r):
    """The definition restated with rationals: t_j = max(0, 1 - |j + 1/2 - c| / sigma)."""
    sigma = max(Fraction(1), Fraction(n_in, r))
    got = aa.axis_weights(n_in, r, 0, r)
    for x in range(r):
        c = Fraction(2 * x + 1, 2) * Fraction(n_in, r)
        t = [max(Fraction(0), 1 - abs(Fraction(2 * j + 1, 2) - c) / sigma) for j in range(n_in)]
        total = sum(t)
        want = np.array([float(v / total) for v in t])
        assert np.allclose(got[x], want, atol=1e-14)
        assert abs(got[x].sum() - 1.0) < 1e-14


def test_first_and_count_select_rows():
    full = aa.axis_weights(50, 12, 0, 12)
    assert np.array_equal(aa.axis_weights(50, 12, 5, 4), full[5:9])


# ---- the resized window ---------------------------------------------------------------------------

def test_resized_size_is_the_plain_transform_s():
    for h, w, s in [(1080, 1920, 256), (375, 500, 256), (500, 375, 256), (7, 7, 3), (100, 333, 17)]:
        assert aa.resized_size(h, w, s) == oracle.resized_size(h, w, s)


def test_constant_image_stays_constant():
    img = np.empty((45, 70, 3), dtype=np.uint8)
    img[..., 0], img[..., 1], img[..., 2] = 7, 200, 255
    v = aa.resized_window(img, 9, 11)
    for ch, val in enumerate((7, 200, 255)):
        assert np.allclose(v[..., ch], val, atol=1e-11)


def test_integer_reduction_reproduces_a_ramp_in_the_interior():
    """p = a + b*j along x, reduced by 4: a symmetric normalised kernel returns the ramp at the
    output's centre, a + b*(4X + 3/2) (pixel j's centre is j + 1/2, so the value at c is
    a + b*(c - 1/2))."""
    a, b, n = 3, 1, 64
    row = (a + b * np.arange(n)).astype(np.uint8)
    img = np.repeat(np.broadcast_to(row[None, :, None], (n, n, 1)), 3, axis=2).copy()
    v = aa.resized_window(img, 16, 16)
    want = a + b * (4 * np.arange(16) + 1.5)
    assert np.allclose(v[5, 2:14, 1], want[2:14], atol=1e-11)
    vt = aa.resized_window(np.ascontiguousarray(np.transpose(img, (1, 0, 2))), 16, 16)
    assert np.allclose(vt[2:14, 7, 2], want[2:14], atol=1e-11)


def test_a_single_bright_pixel_spreads_as_the_product_of_the_two_triangles():
    """8 x 16 image, s = 4: R = 4 x 8, both axes halved.  A pixel of 240 at (row 3, column 6):
    row 3 has weight 3/8 in Y = 1 (pixels 1..4 -> 1/8,3/8,3/8,1/8) and 1/8 in Y = 2 (pixels 3..6);
    column 6 has weight 3/8 in X = 3 (pixels 5..8) and 1/8 in X = 2 (pixels 3..6)."""
    img = np.zeros((8, 16, 3), dtype=np.uint8)
    img[3, 6, 1] = 240
    v = aa.resized_window(img, 4, 4, 0, 1)          # window columns 1..4 of the 4 x 8 grid
    want = np.zeros((4, 4))
    want[1, 2], want[1, 1], want[2, 2], want[2, 1] = 240 * 9 / 64, 240 * 3 / 64, 240 * 3 / 64, 240 / 64
    assert np.allclose(v[..., 1], want, atol=1e-12)
    assert np.all(v[..., 0] == 0) and np.all(v[..., 2] == 0)


@pytest.mark.parametrize("seed,h,w,c,s,origin", [
    (1, 9, 14, 3, 4, None), (2, 14, 9, 4, 4, (1, 0)), (3, 11, 11, 2, 5, (3, 2)),
    (4, 5, 23, 3, 3, (0, 9)), (5, 6, 8, 7, 7, None), (6, 1, 1, 2, 2, None),
])
def test_window_against_exact_fraction_brute_force(seed, h, w, c, s, origin):
    img = rand_img(seed, h, w)
    rh, rw = oracle.resized_size(h, w, s)
    top, left = origin if origin is not None else ((rh - c) // 2, (rw - c) // 2)

    def weights(n_in, r, x):
        sigma = max(Fraction(1), Fraction(n_in, r))
        cen = Fraction(2 * x + 1, 2) * Fraction(n_in, r)
        t = [max(Fraction(0), 1 - abs(Fraction(2 * j + 1, 2) - cen) / sigma) for j in range(n_in)]
        tot = sum(t)
        return [v / tot for v in t]

    got = aa.resized_window(img, c, s, *(origin if origin is not None else (None, None)))
    for k in range(c):
        wy = weights(h, rh, top + k)
        for q in range(c):
            wx = weights(w, rw, left + q)
            for ch in range(3):
                v = sum(wy[i] * wx[j] * int(img[i, j, ch]) for i in range(h) for j in range(w)
                        if wy[i] and wx[j])
                assert abs(got[k, q, ch] - float(v)) < 1e-10


@pytest.mark.parametrize("h,w,s", [(97, 160, 24), (160, 97, 24), (64, 64, 64), (40, 55, 64)])
def test_whole_resized_image_against_the_library_routine(h, w, s):
    """torch's antialiased bilinear interpolation (CPU, float64, half-pixel centres) over the
    whole resized grid; windows at several origins must be its sub-windows."""
    import torch
    import torch.nn.functional as F

    img = rand_img(h * 1000 + w, h, w)
    rh, rw = oracle.resized_size(h, w, s)
    t = torch.from_numpy(img.astype(np.float64)).permute(2, 0, 1)[None]
    ref = F.interpolate(t, size=(rh, rw), mode="bilinear", align_corners=False, antialias=True)
    ref = ref[0].permute(1, 2, 0).numpy()
    c = min(rh, rw) - 3
    for top, left in [(0, 0), (rh - c, rw - c), (1, 2), ((rh - c) // 2, (rw - c) // 2)]:
        got = aa.resized_window(img, c, s, top, left)
        assert np.max(np.abs(got - ref[top:top + c, left:left + c])) < 1e-9
    centre = aa.resized_window(img, c, s)
    assert np.array_equal(centre, aa.resized_window(img, c, s, (rh - c) // 2, (rw - c) // 2))


def test_transposing_the_image_transposes_the_result():
    img = rand_img(8, 50, 81)
    a = aa.resized_window(img, 10, 12)
    b = aa.resized_window(np.ascontiguousarray(np.transpose(img, (1, 0, 2))), 10, 12)
    assert np.allclose(a, np.transpose(b, (1, 0, 2)), atol=1e-11)
    assert not np.allclose(a, b, atol=1e-3)


# ---- the whole transform --------------------------------------------------------------------------

def test_images_that_are_not_reduced_match_the_plain_transform():
    """Both axes enlarged (sigma = 1 on each): the plain oracle's two-tap interpolation."""
    imgs = [rand_img(9, 20, 31), rand_img(10, 33, 17), rand_img(11, 40, 40)]
    c, s = 36, 40
    got = aa.preprocess(imgs, c, s, MEAN, STD)
    want = oracle.preprocess(imgs, c, s, MEAN, STD)
    assert np.max(np.abs(got - want)) < 1e-11


def test_reduced_images_differ_from_the_plain_transform():
    img = rand_img(12, 200, 300)
    got = aa.preprocess([img], 24, 28, MEAN, STD)
    plain = oracle.preprocess([img], 24, 28, MEAN, STD)
    assert np.max(np.abs(got - plain)) > 0.1
    # averaging over ~7 x 7 pixels of white noise shrinks the spread
    assert got.std() < 0.5 * plain.std()


def test_normalisation_and_layout():
    img = np.empty((30, 50, 3), dtype=np.uint8)
    img[..., 0], img[..., 1], img[..., 2] = 0, 128, 255
    out = aa.preprocess([img, img], 8, 10, MEAN, STD, crop_origin=[(0, 0), (2, 8)])
    assert out.shape == (2, 3, 8, 8)
    for ch, val in enumerate((0.0, 128.0, 255.0)):
        want = (val / 255.0 - M64[ch]) / S64[ch]
        assert np.allclose(out[:, ch], want, atol=1e-12)


def test_batch_position_and_origin():
    imgs = [rand_img(20 + i, 60 + 7 * i, 90 - 5 * i) for i in range(4)]
    c, s = 12, 16
    origins = [(i, i + 1) for i in range(4)]
    whole = aa.preprocess(imgs, c, s, MEAN, STD, crop_origin=origins)
    for i, im in enumerate(imgs):
        v = aa.resized_window(im, c, s, *origins[i])
        want = np.transpose((v / 255.0 - M64) / S64, (2, 0, 1))
        assert np.array_equal(whole[i], want)
    with pytest.raises(ValueError):
        aa.preprocess(imgs[:1], c, s, MEAN, STD, crop_origin=[(5, 0)])   # 5 + 12 > 16


# ---- the benchmark's byte accounting (host logic of the package, checked against the oracle) ------

def test_accounting_counts_the_rectangle_of_weighted_pixels():
    from paper_2411_19114_b200 import accounting as ac

    table = np.zeros(3, dtype=[("offset", "<u8"), ("h", "<u4"), ("w", "<u4")])
    sizes = [(1080, 1920), (375, 500), (100, 150)]
    c, s = 224, 256
    want_in = 0
    for t, (h, w) in zip(table, sizes):
        t["h"], t["w"] = h, w
        rh, rw = aa.resized_size(h, w, s)
        rows = np.nonzero(aa.axis_weights(h, rh, (rh - c) // 2, c).sum(axis=0) > 1e-15)[0]
        cols = np.nonzero(aa.axis_weights(w, rw, (rw - c) // 2, c).sum(axis=0) > 1e-15)[0]
        want_in += 3 * (rows[-1] - rows[0] + 1) * (cols[-1] - cols[0] + 1)
    got = ac.antialias_batch_bytes(table, c, s, 4)
    assert got["input_bytes"] == want_in
    assert got["output_bytes"] == 3 * 3 * c * c * 4 and got["total"] == want_in + got["output_bytes"]
