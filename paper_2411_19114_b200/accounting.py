"""Byte accounting for the roofline: what one batch must move through HBM.

Input bytes are counted sector-granular: 32 bytes for every distinct 32-byte-aligned
sector of the packed buffer that holds at least one byte of a tapped source pixel
(tapped = one of the 2x2 bilinear neighbours of some output element).  Output bytes are
the dense result.  This is bookkeeping for the benchmark, not part of the transform.
"""
from __future__ import annotations

import numpy as np

SECTOR = 32


def _taps(n_in: int, r: int, c: int) -> np.ndarray:
    """Sorted distinct source indices tapped along one axis (exact integer geometry)."""
    origin = (r - c) // 2
    X = np.arange(c, dtype=np.int64) + origin
    den = 2 * r
    num = np.clip((2 * X + 1) * n_in - r, 0, (n_in - 1) * den)
    i0 = num // den
    i1 = np.minimum(i0 + 1, n_in - 1)
    # the second tap carries weight only when the remainder is non-zero, but a kernel
    # cannot know that before reading the geometry; both taps count as tapped
    return np.unique(np.concatenate([i0, i1]))


def resized(h: int, w: int, s: int) -> tuple[int, int]:
    return (s, s * w // h) if h <= w else (s * h // w, s)


def image_input_bytes(offset: int, h: int, w: int, c: int, s: int) -> tuple[int, int]:
    """(sector-granular bytes, pixel-exact bytes) of one image's tapped footprint."""
    rh, rw = resized(h, w, s)
    ys, xs = _taps(h, rh, c), _taps(w, rw, c)
    first = offset + 3 * (ys[:, None] * w + xs[None, :])   # first byte of each tapped pixel
    sectors = np.unique(np.concatenate([(first // SECTOR).ravel(), ((first + 2) // SECTOR).ravel()]))
    return int(sectors.size) * SECTOR, 3 * int(ys.size) * int(xs.size)


def batch_bytes(table, c: int, s: int, out_itemsize: int) -> dict:
    """Algorithmic bytes of one launch over the batch described by ``table``
    (records with fields offset, h, w)."""
    a_in = a_px = 0
    for e in table:
        sec, px = image_input_bytes(int(e["offset"]), int(e["h"]), int(e["w"]), c, s)
        a_in += sec
        a_px += px
    a_out = len(table) * 3 * c * c * out_itemsize
    return dict(input_sector_bytes=a_in, input_pixel_bytes=a_px, output_bytes=a_out,
                total=a_in + a_out)


def _support(n_in: int, r: int, first: int, count: int) -> tuple[int, int]:
    """[lo, hi): input pixels that carry weight in some resized pixel first .. first+count-1 of
    the antialiased Resize: |(2j+1) r - (2X+1) n_in| < 2 max(n_in, r), inside the image."""
    m2 = 2 * max(n_in, r)
    lo_c = (2 * first + 1) * n_in
    hi_c = (2 * (first + count - 1) + 1) * n_in
    lo = max(0, (lo_c - m2 - r) // (2 * r) + 1)
    hi = min(n_in, -(-(hi_c + m2 - r) // (2 * r)))
    return lo, hi


def antialias_batch_bytes(table, c: int, s: int, out_itemsize: int) -> dict:
    """Bytes one antialiased batch must move through HBM: every byte of the rectangle of
    input pixels under the centre crop's support, once, plus the dense output."""
    inp = 0
    for t in table:
        h, w = int(t["h"]), int(t["w"])
        rh, rw = resized(h, w, s)
        y0, y1 = _support(h, rh, (rh - c) // 2, c)
        x0, x1 = _support(w, rw, (rw - c) // 2, c)
        inp += 3 * (y1 - y0) * (x1 - x0)
    out = len(table) * 3 * c * c * out_itemsize
    return {"input_bytes": inp, "output_bytes": out, "total": inp + out}
