"""GPU parity of preba_preprocess_antialias against the antialias oracle (float64), element by
element.  Tolerance for fp32 output: both sides sum at most a few hundred products of
normalised weights and values below 256; the kernel's fp32 weights and sums are each within a
few 2^-24 relative, so the resized value is within about 1e-4 of 255 and the normalised one
(multiplied by 1/(255*std) < 0.02) within 2e-6; the tests allow 1e-5, the plain path's bound.
fp16 and bf16 outputs are held to the plain path's criteria (helpers.assert_parity)."""
from __future__ import annotations

import numpy as np
import pytest

from helpers import MEAN, STD, assert_parity
from oracle import antialias as aa
from paper_2411_19114_b200 import binding as pb
from paper_2411_19114_b200 import workloads as wl

pytestmark = pytest.mark.gpu

GUARD, CANARY = 4096, 0xA5
ITEM = {pb.F32: 4, pb.F16: 2, pb.BF16: 2}
VIEW = {pb.F32: np.float32, pb.F16: np.float16, pb.BF16: np.uint16}


def uniform(seed, h, w):
    return wl.uniform_image(np.random.default_rng(seed), h, w)


def run(images, c, s, out_dtype=pb.F32, origins=None, with_host_table=True, expect_status=0):
    import torch

    n = len(images)
    packed, table = pb.preba_pack(images)
    dev = torch.device("cuda:0")
    ob = n * 3 * c * c * ITEM[out_dtype]
    out_buf = torch.full((GUARD + ob + GUARD,), CANARY, dtype=torch.uint8, device=dev)
    out = out_buf[GUARD:GUARD + ob]
    pix = torch.from_numpy(packed).to(dev)
    tab = torch.from_numpy(table.view(np.uint8)).to(dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    crop = torch.from_numpy(origins.astype(np.int64)).to(dev).to(torch.int32).reshape(-1) \
        if origins is not None else None
    pb.preba_preprocess_antialias(pix, tab, n, out, c, s, MEAN, STD, out_dtype, crop_origin=crop,
                                  crop_origin_host=origins if with_host_table else None,
                                  table_host=table if with_host_table else None, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == expect_status, pb.preba_strerror(int(status.item()))
    host = out_buf.cpu().numpy()
    assert np.all(host[:GUARD] == CANARY) and np.all(host[GUARD + ob:] == CANARY), \
        "kernel wrote outside the output tensor"
    return host[GUARD:GUARD + ob].copy().view(VIEW[out_dtype]).reshape(n, 3, c, c)


def want(images, c, s, origins=None):
    o = None if origins is None else [tuple(int(v) for v in r) for r in origins]
    return aa.preprocess(images, c, s, MEAN, STD, crop_origin=o)


def origins_for(images, c, s, seed):
    rng = np.random.default_rng(seed)
    out = []
    for i, im in enumerate(images):
        rh, rw = aa.resized_size(im.shape[0], im.shape[1], s)
        corner = i % 5
        top = [0, rh - c, 0, rh - c, int(rng.integers(0, rh - c + 1))][corner]
        left = [0, 0, rw - c, rw - c, int(rng.integers(0, rw - c + 1))][corner]
        out.append((top, left))
    return np.asarray(out, dtype=np.uint32)


# reduced a lot, a little, not at all, enlarged; pitches of every residue modulo 4
SHAPES = [(1080, 1920), (700, 901), (375, 500), (500, 375), (241, 499), (256, 256), (257, 342),
          (100, 150), (903, 602), (1200, 1203), (64, 2000), (2000, 65)]


def test_ragged_batch_fp32_centre_crop():
    images = [uniform(100 + i, h, w) for i, (h, w) in enumerate(SHAPES)]
    got = run(images, 224, 256)
    ref = want(images, 224, 256)
    err = np.max(np.abs(got - ref), axis=(1, 2, 3))
    assert np.all(err <= 1e-5), err


# widths that are multiples of 4 (rows start on the same byte phase: the images the
# tensor-core kernel takes), with row pitches of every residue modulo 16, reduced up to 5 times,
# not at all, and enlarged
MMA_SHAPES = [(1080, 1920), (771, 1028), (600, 808), (333, 444), (250, 1000), (900, 400),
              (256, 256), (1280, 1284), (120, 160), (517, 1372)]


@pytest.mark.parametrize("c,s", [(224, 256), (100, 130), (65, 65), (33, 300), (288, 320)])
def test_images_of_the_tensor_core_kernel(c, s):
    images = [uniform(150 + i, h, w) for i, (h, w) in enumerate(MMA_SHAPES)]
    got = run(images, c, s)
    err = np.max(np.abs(got - want(images, c, s)), axis=(1, 2, 3))
    assert np.all(err <= 1e-5), err
    origins = origins_for(images, c, s, 11)
    got = run(images, c, s, origins=origins, with_host_table=False)
    err = np.max(np.abs(got - want(images, c, s, origins)), axis=(1, 2, 3))
    assert np.all(err <= 1e-5), err


# images reduced between 2.5 and about 6.5 times vertically, widths that are multiples of 4: the
# ones that take both passes on the tensor cores (windows of three and of four steps, groups
# with a ragged last tile, portrait and landscape), next to some that just miss it
CHAINED_SHAPES = [(1080, 1920), (700, 1000), (1600, 1600), (650, 2000), (1920, 1080), (1000, 1404),
                  (1284, 1280), (644, 644), (1700, 1704), (640, 1640)]


@pytest.mark.parametrize("c,s", [(224, 256), (256, 256), (75, 240), (76, 250), (33, 300), (1, 200)])
def test_images_of_the_chained_tensor_core_kernel(c, s):
    images = [uniform(170 + i, h, w) for i, (h, w) in enumerate(CHAINED_SHAPES)]
    got = run(images, c, s)
    err = np.max(np.abs(got - want(images, c, s)), axis=(1, 2, 3))
    assert np.all(err <= 1e-5), err
    origins = origins_for(images, c, s, 13)
    got = run(images, c, s, origins=origins, with_host_table=False)
    err = np.max(np.abs(got - want(images, c, s, origins)), axis=(1, 2, 3))
    assert np.all(err <= 1e-5), err
    # one image alone: its rows are cut into CTAs differently, but the tiles of input rows sit
    # at the same places of the image, so the sums group their terms alike
    alone = run(images[:1], c, s)
    assert np.array_equal(alone[0], run(images, c, s)[0])


@pytest.mark.parametrize("out_dtype", [pb.F16, pb.BF16])
def test_half_precision_outputs_of_the_chained_kernel(out_dtype):
    images = [wl.smooth_image(np.random.default_rng(470 + i), h, w)
              for i, (h, w) in enumerate(CHAINED_SHAPES[:5])]
    got = run(images, 224, 256, out_dtype=out_dtype)
    assert_parity(got, want(images, 224, 256), out_dtype)


@pytest.mark.parametrize("c,s", [(224, 256), (96, 96), (17, 40), (1, 1), (299, 342)])
def test_other_output_sizes(c, s):
    images = [uniform(200 + i, h, w) for i, (h, w) in enumerate(SHAPES[:7])]
    got = run(images, c, s)
    assert np.max(np.abs(got - want(images, c, s))) <= 1e-5


def test_crop_windows_per_image():
    images = [uniform(300 + i, h, w) for i, (h, w) in enumerate(SHAPES)]
    origins = origins_for(images, 160, 256, 7)
    got = run(images, 160, 256, origins=origins)
    assert np.max(np.abs(got - want(images, 160, 256, origins))) <= 1e-5
    # and without the host copies (the launch then carries all the shared memory there is)
    got2 = run(images, 160, 256, origins=origins, with_host_table=False)
    assert np.array_equal(got, got2)


@pytest.mark.parametrize("out_dtype", [pb.F16, pb.BF16])
def test_half_precision_outputs(out_dtype):
    images = [wl.smooth_image(np.random.default_rng(400 + i), h, w)
              for i, (h, w) in enumerate(SHAPES[:8])]
    got = run(images, 224, 256, out_dtype=out_dtype)
    assert_parity(got, want(images, 224, 256), out_dtype)


def test_degenerate_images():
    images = [uniform(500, 1, 1), uniform(501, 1, 40), uniform(502, 40, 1), uniform(503, 2, 3000),
              uniform(504, 3000, 2), uniform(505, 5, 5)]
    got = run(images, 4, 4)
    assert np.max(np.abs(got - want(images, 4, 4))) <= 1e-5


def test_enlargements_whose_integer_weights_pass_16_bits_take_the_fp32_path():
    """300 x 4 and 4 x 300 at resize_short = 16384: one axis is enlarged to 1,228,800 pixels, so
    its un-normalised weights need 22 bits; the vertical pass then sums in fp32."""
    images = [uniform(550, 300, 4), uniform(551, 4, 300), uniform(552, 7, 5)]
    got = run(images, 8, 16384)
    assert np.max(np.abs(got - want(images, 8, 16384))) <= 1e-5
    origins = np.asarray([[1228800 - 8, 16384 - 8], [0, 1228800 - 8], [11, 3]], dtype=np.uint32)
    got = run(images, 8, 16384, origins=origins)
    assert np.max(np.abs(got - want(images, 8, 16384, origins))) <= 1e-5


def test_small_batches_take_fewer_rows_per_block():
    """One image: the launch splits it into single rows; the result does not depend on it."""
    img = uniform(600, 1080, 1920)
    alone = run([img], 224, 256)
    among = run([uniform(601 + i, 300, 400) for i in range(40)] + [img], 224, 256)
    assert np.array_equal(alone[0], among[-1])
    assert np.max(np.abs(alone - want([img], 224, 256))) <= 1e-5


def test_images_that_are_not_reduced_match_the_plain_entry_point():
    import torch

    images = [uniform(700 + i, h, w) for i, (h, w) in enumerate([(100, 150), (200, 130), (224, 224)])]
    got = run(images, 224, 256)
    packed, table = pb.preba_pack(images)
    dev = torch.device("cuda:0")
    out = torch.empty((3, 3, 224, 224), dtype=torch.float32, device=dev)
    pb.preba_preprocess(torch.from_numpy(packed).to(dev), torch.from_numpy(table.view(np.uint8)).to(dev),
                        3, out, 224, 256, MEAN, STD, pb.F32, table_host=table)
    torch.cuda.synchronize()
    assert np.max(np.abs(got - out.cpu().numpy())) <= 4e-6


def test_full_size_batch_of_the_bench():
    """64 frames of 1080 x 1920 (the batch the bench times), every element."""
    images = wl.hires_1080p(64, seed=800)
    got = run(images, 224, 256)
    ref = want(images, 224, 256)
    assert np.max(np.abs(got - ref)) <= 1e-5


# ---- refusals -------------------------------------------------------------------------------------

def _call(images, c, s, **kw):
    import torch

    packed, table = pb.preba_pack(images)
    dev = torch.device("cuda:0")
    out = torch.zeros(len(images) * 3 * c * c, dtype=torch.float32, device=dev)
    pix = torch.from_numpy(packed).to(dev)
    tab = torch.from_numpy(table.view(np.uint8)).to(dev)
    pb.preba_preprocess_antialias(pix, tab, len(images), out, c, s, MEAN, STD, pb.F32,
                                  table_host=table, **kw)
    torch.cuda.synchronize()


def test_bad_arguments_are_refused():
    images = [uniform(900, 30, 40)]
    with pytest.raises(pb.PrebaError) as e:
        _call(images, 20, 10)                      # crop larger than the resized shorter side
    assert e.value.code == pb.ERR_INVALID_ARG
    with pytest.raises(pb.PrebaError) as e:
        _call(images, 8, 10, crop_origin_host=np.asarray([[3, 0]], dtype=np.uint32))
    assert e.value.code == pb.ERR_BAD_CROP


def test_a_window_off_the_grid_is_skipped_and_reported_by_the_kernel():
    images = [uniform(901, 30, 40), uniform(902, 50, 50)]
    origins = np.asarray([[3, 0], [0, 0]], dtype=np.uint32)     # 3 + 8 > 10 for the first image
    got = run(images, 8, 10, origins=origins, with_host_table=False,
              expect_status=pb.ERR_BAD_CROP)
    assert np.all(got[0].view(np.uint8) == CANARY)              # untouched
    assert np.max(np.abs(got[1] - want(images[1:], 8, 10, origins[1:])[0])) <= 1e-5


def test_an_image_reduced_beyond_the_working_set_is_refused():
    """One 11,601 x 11,601 image at out_size = resize_short = 2,320 needs more shared memory
    than a block can have (its width is not a multiple of 4, so the tensor-core kernel, which
    works on column groups and needs far less, does not take it): refused on the host with the
    table, reported by the kernel without."""
    import torch

    side, c = 11601, 2320
    dev = torch.device("cuda:0")
    pix = torch.zeros(3 * side * side + 128, dtype=torch.uint8, device=dev)
    table = np.zeros(1, dtype=pb.TABLE_DTYPE)
    table["h"], table["w"] = side, side
    tab = torch.from_numpy(table.view(np.uint8)).to(dev)
    out = torch.full((3 * c * c,), 7.0, dtype=torch.float32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    with pytest.raises(pb.PrebaError) as e:
        pb.preba_preprocess_antialias(pix, tab, 1, out, c, c, MEAN, STD, pb.F32, table_host=table)
    assert e.value.code == pb.ERR_TOO_LARGE
    pb.preba_preprocess_antialias(pix, tab, 1, out, c, c, MEAN, STD, pb.F32, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == pb.ERR_TOO_LARGE
    assert bool(torch.all(out == 7.0))


def test_a_large_image_of_the_tensor_core_kernel():
    """11,600 x 2,000 pixels reduced five times to 2,320 x 400, crop 400: column groups and
    bands beyond the first, rows far apart in memory."""
    images = [uniform(950, 2000, 11600)]
    got = run(images, 400, 400)
    assert np.max(np.abs(got - want(images, 400, 400))) <= 1e-5
