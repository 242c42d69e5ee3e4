"""GPU parity of preba_preprocess_ex (crop window per image, rounding to uint8) against the
variant oracle: uint8 output bit for bit, float outputs within the criteria of the base path."""
from __future__ import annotations

import numpy as np
import pytest

import oracle
from helpers import MEAN, STD, assert_parity, host_threads
from paper_2411_19114_b200 import binding as pb
from paper_2411_19114_b200 import workloads as wl

pytestmark = pytest.mark.gpu

GUARD, CANARY = 4096, 0xA5


def uniform(seed, h, w):
    return wl.uniform_image(np.random.default_rng(seed), h, w)


def origins_for(images, c, s, seed):
    """A window per image, drawn over the whole range the resized grid allows (corners too)."""
    rng = np.random.default_rng(seed)
    out = []
    for i, im in enumerate(images):
        rh, rw = oracle.resized_size(im.shape[0], im.shape[1], s)
        corner = i % 5
        top = [0, rh - c, 0, rh - c, int(rng.integers(0, rh - c + 1))][corner]
        left = [0, 0, rw - c, rw - c, int(rng.integers(0, rw - c + 1))][corner]
        out.append((top, left))
    return np.asarray(out, dtype=np.uint32)


def run_ex(images, c, s, out_dtype, round_u8, origins=None, mean=MEAN, std=STD, dynamic=True):
    import torch

    n = len(images)
    packed, table = pb.preba_pack(images)
    dev = torch.device("cuda:0")
    item = {pb.F32: 4, pb.F16: 2, pb.BF16: 2, pb.U8: 1}[out_dtype]
    ob = n * 3 * c * c * item
    out_buf = torch.full((GUARD + ob + GUARD,), CANARY, dtype=torch.uint8, device=dev)
    out = out_buf[GUARD:GUARD + ob]
    pix = torch.from_numpy(packed).to(dev)
    tab = torch.from_numpy(table.view(np.uint8)).to(dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    scratch = torch.zeros(pb.SCRATCH_BYTES // 4, dtype=torch.int32, device=dev) if dynamic else None
    crop = torch.from_numpy(origins.astype(np.int64)).to(dev).to(torch.int32).reshape(-1) \
        if origins is not None else None
    pb.preba_preprocess_ex(pix, tab, n, out, c, s, mean, std, out_dtype, round_u8=round_u8,
                           crop_origin=crop, crop_origin_host=origins, table_host=table,
                           status=status, scratch=scratch)
    torch.cuda.synchronize()
    assert int(status.item()) == 0, pb.preba_strerror(int(status.item()))
    host = out_buf.cpu().numpy()
    assert np.all(host[:GUARD] == CANARY) and np.all(host[GUARD + ob:] == CANARY), \
        "kernel wrote outside the output tensor"
    res = host[GUARD:GUARD + ob].copy()
    if out_dtype == pb.U8:
        return res.reshape(n, c, c, 3)
    view = {pb.F32: np.float32, pb.F16: np.float16, pb.BF16: np.uint16}[out_dtype]
    return res.view(view).reshape(n, 3, c, c)


def want_u8(images, c, s, origins):
    return oracle.preprocess_ex(images, c, s, MEAN, STD, oracle.OUT_U8_HWC, crop_origin=origins,
                                round_u8=True, nthreads=host_threads())


def want_f64(images, c, s, origins, round_u8, mean=MEAN, std=STD):
    return oracle.preprocess_ex(images, c, s, mean, std, oracle.OUT_F64, crop_origin=origins,
                                round_u8=round_u8, nthreads=host_threads())


SHAPES = [(240, 320), (375, 500), (500, 375), (241, 499), (500, 240), (256, 256), (333, 257)]


@pytest.mark.parametrize("dynamic", [True, False])
def test_uint8_output_is_bit_exact_on_a_ragged_batch(dynamic):
    imgs = [uniform(40 + i, h, w) for i, (h, w) in enumerate(SHAPES)] + wl.mixed_smooth(6, seed=41)
    for origins in (None, origins_for(imgs, 224, 256, 1)):
        got = run_ex(imgs, 224, 256, pb.U8, True, origins, dynamic=dynamic)
        assert np.array_equal(got, want_u8(imgs, 224, 256, origins))


@pytest.mark.parametrize("c,s", [(1, 1), (7, 7), (9, 17), (33, 40), (224, 224), (225, 300), (449, 460),
                                 (40, 800), (230, 1000)])  # the last two: division with correction
def test_uint8_output_other_sizes_and_partial_column_blocks(c, s):
    imgs = [uniform(50, 37, 53), uniform(51, 64, 48), uniform(52, 5, 9), uniform(53, 300, 200)]
    origins = origins_for(imgs, c, s, 2)
    got = run_ex(imgs, c, s, pb.U8, True, origins)
    assert np.array_equal(got, want_u8(imgs, c, s, origins))


def test_uint8_identity_and_ties():
    """H = W = S = C gives the image back; a two-times upscale of an even ramp is all ties."""
    img = uniform(54, 224, 224)
    assert np.array_equal(run_ex([img], 224, 224, pb.U8, True)[0], img)
    n = 112
    row = (2 * np.arange(n) % 256).astype(np.uint8)
    ramp = np.repeat(np.broadcast_to(row[None, :, None], (n, n, 1)), 3, axis=2).copy()
    got = run_ex([ramp], 224, 224, pb.U8, True)
    assert np.array_equal(got, want_u8([ramp], 224, 224, None))


def test_uint8_exact_path_for_sizes_beyond_32_bit_products():
    """A strong upscale (den products beyond 2^32 / 511) and a 13x downscale take the exact
    wide-integer path; so does a 2 x 32768 strip."""
    imgs = [uniform(55, 40, 30), uniform(56, 3000, 2900), uniform(57, 2, 32768)]
    c, s = 40, 2000
    origins = np.asarray([(0, 0), (100, 37)], dtype=np.uint32)
    got = run_ex(imgs[:2], c, s, pb.U8, True, origins)
    assert np.array_equal(got, want_u8(imgs[:2], c, s, origins))
    strip = np.asarray([(0, 50001)], dtype=np.uint32)
    got = run_ex(imgs[2:], 7, 7, pb.U8, True, strip)
    assert np.array_equal(got, want_u8(imgs[2:], 7, 7, strip))


@pytest.mark.parametrize("dt", [pb.F32, pb.F16, pb.BF16])
def test_rounded_then_normalised(dt):
    imgs = [uniform(60 + i, h, w) for i, (h, w) in enumerate(SHAPES[:5])] + wl.mixed_smooth(3, seed=61)
    origins = origins_for(imgs, 224, 256, 3)
    got = run_ex(imgs, 224, 256, dt, True, origins)
    assert_parity(got, want_f64(imgs, 224, 256, origins, True), dt)


@pytest.mark.parametrize("dt", [pb.F32, pb.F16])
def test_crop_window_per_image_without_rounding(dt):
    imgs = [uniform(70 + i, h, w) for i, (h, w) in enumerate(SHAPES)] + wl.mixed_smooth(4, seed=71)
    origins = origins_for(imgs, 224, 256, 4)
    got = run_ex(imgs, 224, 256, dt, False, origins)
    assert_parity(got, want_f64(imgs, 224, 256, origins, False), dt)
    # the centre window given explicitly is the centre crop of the plain entry point, bit for bit
    centre = np.asarray([((oracle.resized_size(*im.shape[:2], 256)[0] - 224) // 2,
                          (oracle.resized_size(*im.shape[:2], 256)[1] - 224) // 2) for im in imgs],
                        dtype=np.uint32)
    a = run_ex(imgs, 224, 256, dt, False, centre)
    b = run_ex(imgs, 224, 256, dt, False, None)
    assert np.array_equal(a.view(np.uint8), b.view(np.uint8))


def test_full_mixed_workload_uint8():
    imgs = wl.mixed_smooth(256, seed=2)
    got = run_ex(imgs, wl.OUT_SIZE, wl.RESIZE_SHORT, pb.U8, True)
    assert np.array_equal(got, want_u8(imgs, wl.OUT_SIZE, wl.RESIZE_SHORT, None))


def test_window_outside_the_resized_image_is_refused_or_skipped():
    import torch

    imgs = [uniform(80, 240, 320), uniform(81, 240, 320)]
    n = len(imgs)
    packed, table = pb.preba_pack(imgs)
    dev = torch.device("cuda:0")
    pix = torch.from_numpy(packed).to(dev)
    tab = torch.from_numpy(table.view(np.uint8)).to(dev)
    out = torch.full((n, 224, 224, 3), 7, dtype=torch.uint8, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    bad = np.asarray([(0, 0), (33, 0)], dtype=np.uint32)          # 33 + 224 > 256
    crop = torch.from_numpy(bad.astype(np.int64)).to(dev).to(torch.int32).reshape(-1)
    with pytest.raises(pb.PrebaError) as exc:                     # host copies given: refused
        pb.preba_preprocess_ex(pix, tab, n, out, 224, 256, MEAN, STD, pb.U8, round_u8=True,
                               crop_origin=crop, crop_origin_host=bad, table_host=table,
                               status=status)
    assert exc.value.code == pb.ERR_BAD_CROP
    # without them the kernel finds it: that image is skipped, the other is computed
    pb.preba_preprocess_ex(pix, tab, n, out, 224, 256, MEAN, STD, pb.U8, round_u8=True,
                           crop_origin=crop, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == pb.ERR_BAD_CROP
    host = out.cpu().numpy()
    assert np.all(host[1] == 7)
    assert np.array_equal(host[0], want_u8(imgs[:1], 224, 256, bad[:1])[0])


@pytest.mark.parametrize("seed", range(6))
def test_random_shapes_windows_and_modes(seed):
    """Seeded random batches: sides from 1 to 700, random crop and resize sizes, a random
    window per image, all modes.  uint8 bit for bit; float kinds by the base criteria."""
    rng = np.random.default_rng(9000 + seed)
    s_short = int(rng.integers(1, 400))
    c = int(rng.integers(1, s_short + 1))
    n = int(rng.integers(1, 10))
    imgs = [wl.uniform_image(rng, int(rng.integers(1, 701)), int(rng.integers(1, 701)))
            for _ in range(n)]
    origins = origins_for(imgs, c, s_short, 100 + seed) if seed % 3 else None
    dynamic = bool(seed & 1)
    got = run_ex(imgs, c, s_short, pb.U8, True, origins, dynamic=dynamic)
    assert np.array_equal(got, want_u8(imgs, c, s_short, origins))
    for dt in (pb.F32, pb.F16, pb.BF16):
        got = run_ex(imgs, c, s_short, dt, True, origins, dynamic=dynamic)
        assert_parity(got, want_f64(imgs, c, s_short, origins, True), dt)
    if origins is not None:
        got = run_ex(imgs, c, s_short, pb.F32, False, origins, dynamic=dynamic)
        assert_parity(got, want_f64(imgs, c, s_short, origins, False), pb.F32)
