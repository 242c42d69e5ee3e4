"""TEST INFRASTRUCTURE ONLY: exact-rational brute force of the preprocessing definition.

For tiny images this evaluates resize -> center crop -> normalise (paper Sec. 2.3
item 1, Table 1 order) with ``fractions.Fraction``, so there is no rounding at
all.  It is written from the continuous statement of bilinear sampling (pixel
centres at half-integers, coordinate clamped to the image), not from the
integer num/den form the C oracle uses, so an indexing slip in either shows up
as a disagreement.  Pure-Python loops: small cases only.
"""
from __future__ import annotations

from fractions import Fraction
from math import floor


def resized_size(h: int, w: int, s: int) -> tuple[int, int]:
    if h <= w:
        return s, (s * w) // h
    return (s * h) // w, s


def sample_coord(n_in: int, r: int, c: int, j: int) -> Fraction:
    """Source coordinate (pixel-index units) of crop index j along one axis."""
    origin = (r - c) // 2
    centre = Fraction(2 * (origin + j) + 1, 2)       # centre of resized pixel, in resized units
    sx = centre * Fraction(n_in, r) - Fraction(1, 2)  # same point in source pixel indices
    return min(max(sx, Fraction(0)), Fraction(n_in - 1))


def bilinear(img, h: int, w: int, sy: Fraction, sx: Fraction, ch: int) -> Fraction:
    """Tent-weighted sum of the (up to) four neighbours of (sy, sx); img[y][x][ch] ints."""
    y0, x0 = floor(sy), floor(sx)
    fy, fx = sy - y0, sx - x0
    y1, x1 = min(y0 + 1, h - 1), min(x0 + 1, w - 1)
    return ((1 - fy) * (1 - fx) * int(img[y0][x0][ch]) + (1 - fy) * fx * int(img[y0][x1][ch])
            + fy * (1 - fx) * int(img[y1][x0][ch]) + fy * fx * int(img[y1][x1][ch]))


def preprocess(img, c: int, s: int, mean, std) -> list:
    """out[ch][k][j] as Fractions for one HWC image (nested lists or array of ints).

    mean/std are taken as the exact values of the given floats."""
    h, w = len(img), len(img[0])
    rh, rw = resized_size(h, w, s)
    assert rh >= c and rw >= c
    mean = [Fraction(float(m)) for m in mean]
    std = [Fraction(float(v)) for v in std]
    ys = [sample_coord(h, rh, c, k) for k in range(c)]
    xs = [sample_coord(w, rw, c, j) for j in range(c)]
    return [[[(bilinear(img, h, w, ys[k], xs[j], ch) / 255 - mean[ch]) / std[ch]
              for j in range(c)] for k in range(c)] for ch in range(3)]


def sample_coord_at(n_in: int, r: int, X: int) -> Fraction:
    """Source coordinate of resized index X along one axis (centre of resized pixel X)."""
    sx = Fraction(2 * X + 1, 2) * Fraction(n_in, r) - Fraction(1, 2)
    return min(max(sx, Fraction(0)), Fraction(n_in - 1))


def resized_pixels(img, c: int, s: int, top: int | None = None, left: int | None = None) -> list:
    """v[k][j][ch] as Fractions: the bilinear value at the c x c window whose first resized
    row/column is (top, left) (centre crop when None), before any rounding or normalisation."""
    h, w = len(img), len(img[0])
    rh, rw = resized_size(h, w, s)
    top = (rh - c) // 2 if top is None else top
    left = (rw - c) // 2 if left is None else left
    assert top + c <= rh and left + c <= rw
    ys = [sample_coord_at(h, rh, top + k) for k in range(c)]
    xs = [sample_coord_at(w, rw, left + j) for j in range(c)]
    return [[[bilinear(img, h, w, ys[k], xs[j], ch) for ch in range(3)]
             for j in range(c)] for k in range(c)]


def round_half_up(v: Fraction) -> int:
    return floor(v + Fraction(1, 2))
