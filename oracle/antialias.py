"""TEST INFRASTRUCTURE ONLY: CPU oracle of the antialiased Resize variant (numpy, float64).

The paper's Resize unit (Table 1) is reconfigured per model "by incremental changes"
(Sec. 4.2, "Flexible design based on reconfigurable hardware"); it fixes no filter.  Reading
taken here for inputs much larger than the model's resolution: the separable triangle
("bilinear") filter whose support grows with the reduction factor, as image libraries apply
when they downscale with antialiasing.  On each axis, with n_in input pixels, R resized pixels,
pixel centres at j + 1/2:

    sigma = max(1, n_in / R)                       half-width of the triangle, in input pixels
    c(X)  = (X + 1/2) * n_in / R                   centre of resized pixel X, in input coordinates
    t_j   = max(0, 1 - |j + 1/2 - c(X)| / sigma)   over the pixels 0 <= j < n_in
    w_j   = t_j / sum_j t_j                        (normalised: borders lose no brightness)

    v[Y][X][ch] = sum_i sum_j wy_i(Y) * wx_j(X) * p[i][j][ch]

followed by the same crop (centre floor((R - C)/2), or an explicit origin) and the same
normalisation (v/255 - mean)/std as the plain transform, mean and std taken as float32.
Where an axis is not reduced (sigma = 1) this is the plain transform's two-tap interpolation
with half-pixel centres and clamped borders.  The resized size is the plain transform's
(shorter side -> S, longer side floor(S*long/short)); each axis uses its own n_in / R.

The definition is written out as two dense weight matrices and two matrix products (the
library step); nothing is blocked or reordered.  The module shares nothing with the CUDA path.
Pinned by tests/test_antialias_oracle_pins.py, whose expected values do not come from it.
"""
from __future__ import annotations

import numpy as np


def resized_size(h: int, w: int, s: int) -> tuple[int, int]:
    """Shorter side -> s, longer side floor(s*long/short)."""
    if h <= w:
        return s, s * w // h
    return s * h // w, s


def axis_weights(n_in: int, r: int, first: int, count: int) -> np.ndarray:
    """[count, n_in]: row q holds the normalised weights of resized pixel first + q."""
    sigma = max(1.0, n_in / r)
    x = np.arange(first, first + count, dtype=np.float64)[:, None]
    j = np.arange(n_in, dtype=np.float64)[None, :]
    centre = (x + 0.5) * n_in / r
    t = np.maximum(0.0, 1.0 - np.abs(j + 0.5 - centre) / sigma)
    return t / t.sum(axis=1, keepdims=True)


def resized_window(img: np.ndarray, c: int, s: int, top: int | None = None,
                   left: int | None = None) -> np.ndarray:
    """[c, c, 3] float64: the antialiased resized image's window at (top, left), 0..255 scale."""
    h, w = img.shape[:2]
    rh, rw = resized_size(h, w, s)
    top = (rh - c) // 2 if top is None else top
    left = (rw - c) // 2 if left is None else left
    if top < 0 or left < 0 or top + c > rh or left + c > rw:
        raise ValueError("crop window outside the resized image")
    wy = axis_weights(h, rh, top, c)
    wx = axis_weights(w, rw, left, c)
    p = img.astype(np.float64)
    out = np.empty((c, c, 3), dtype=np.float64)
    for ch in range(3):
        out[:, :, ch] = wy @ p[:, :, ch] @ wx.T
    return out


def preprocess(images: list[np.ndarray], c: int, s: int, mean, std,
               crop_origin=None) -> np.ndarray:
    """[n, 3, c, c] float64."""
    m = np.asarray(mean, dtype=np.float32).astype(np.float64)
    d = np.asarray(std, dtype=np.float32).astype(np.float64)
    out = np.empty((len(images), 3, c, c), dtype=np.float64)
    for i, img in enumerate(images):
        top, left = (None, None) if crop_origin is None else crop_origin[i]
        v = resized_window(img, c, s, top, left)
        out[i] = np.transpose((v / 255.0 - m) / d, (2, 0, 1))
    return out
