"""The roofline's numerator: `accounting.batch_bytes` against figures worked out apart from it.

The algorithmic input bytes of an image are 32 bytes for every distinct 32-byte sector of the
packed buffer that holds a byte of a tapped pixel (both bilinear neighbours of every output
position count as tapped); the output bytes are the dense result.
"""
import numpy as np
import pytest

import oracle
from paper_2411_19114_b200 import accounting as ac

TABLE = np.dtype([("offset", "<u8"), ("h", "<u4"), ("w", "<u4")])


def one(h, w, offset=0):
    t = np.zeros(1, dtype=TABLE)
    t["offset"], t["h"], t["w"] = offset, h, w
    return t


# Per-image figures of the three fixed-size workloads (resize 256, crop 224, image base on a
# 128-byte boundary), worked out when the workloads were defined: tapped 32-byte sectors.
@pytest.mark.parametrize("h,w,itemsize,a_in,a_out", [
    (240, 320, 4, 135_680, 602_112),
    (375, 500, 2, 335_552, 301_056),
    (1080, 1920, 4, 1_275_904, 602_112),
])
def test_fixed_size_workloads(h, w, itemsize, a_in, a_out):
    got = ac.batch_bytes(one(h, w), 224, 256, itemsize)
    assert got["input_sector_bytes"] == a_in
    assert got["output_bytes"] == a_out
    assert got["total"] == a_in + a_out


def brute_force_sectors(offset, h, w, c, s):
    """Sectors touched by the taps the oracle's own geometry reports, one output position at a
    time, every byte of every tapped pixel marked in a set."""
    rh, rw = oracle.resized_size(h, w, s)
    rows, cols = set(), set()
    for k in range(c):
        y0, y1, _ = oracle.axis(h, rh, c, k)
        rows.update((y0, y1))
    for j in range(c):
        x0, x1, _ = oracle.axis(w, rw, c, j)
        cols.update((x0, x1))
    sectors = set()
    for y in rows:
        for x in cols:
            for b in range(3):
                sectors.add((offset + 3 * (y * w + x) + b) // 32)
    return 32 * len(sectors), 3 * len(rows) * len(cols)


@pytest.mark.parametrize("h,w,c,s,offset", [
    (7, 9, 5, 6, 0), (9, 7, 5, 6, 128), (16, 16, 16, 16, 256), (31, 50, 12, 17, 384),
    (50, 31, 17, 17, 1280), (3, 200, 3, 3, 0), (64, 48, 20, 24, 128 * 37), (1, 1, 1, 1, 0),
    (5, 5, 8, 11, 0),
])
def test_against_brute_force_from_oracle_taps(h, w, c, s, offset):
    want_sec, want_px = brute_force_sectors(offset, h, w, c, s)
    got_sec, got_px = ac.image_input_bytes(offset, h, w, c, s)
    assert (got_sec, got_px) == (want_sec, want_px)


def test_batch_is_the_sum_of_its_images():
    rng = np.random.default_rng(7)
    sizes = [(int(a), int(b)) for a, b in rng.integers(8, 60, size=(6, 2))]
    table = np.zeros(len(sizes), dtype=TABLE)
    at = 0
    for t, (h, w) in zip(table, sizes):
        t["offset"], t["h"], t["w"] = at, h, w
        at = -(-(at + 3 * h * w) // 128) * 128
    c, s = 6, 8
    got = ac.batch_bytes(table, c, s, 2)
    want = sum(brute_force_sectors(int(t["offset"]), int(t["h"]), int(t["w"]), c, s)[0]
               for t in table)
    assert got["input_sector_bytes"] == want
    assert got["output_bytes"] == len(sizes) * 3 * c * c * 2
    assert got["total"] == want + got["output_bytes"]
    # a sector can never be counted for less than the pixels inside it
    assert got["input_pixel_bytes"] <= got["input_sector_bytes"]
