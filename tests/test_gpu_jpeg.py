"""GPU parity of the JPEG Decode unit against its oracle through the C ABI: quantised
coefficients and decoded RGB bytes bit for bit (integer work from the entropy decoder to the
colour conversion: both sides take the same exact-integer inverse transform), the packed layout
and table, the chain into the transform, and the refusals."""
from __future__ import annotations

import ctypes
import io

import numpy as np
import pytest

import oracle
from oracle import jpeg as oj
from paper_2411_19114_b200 import binding as pb
from paper_2411_19114_b200 import workloads as wl

from helpers import MEAN, STD, FP32_TOL, host_threads

GUARD, CANARY = 4096, 0xA5


def decode_on_gpu(jpegs, expect_status=0):
    """(images, quantised coefficients as the device wrote them, table) through preba_jpeg_decode."""
    import torch

    dev = torch.device("cuda:0")
    h, w, sz = pb.preba_jpeg_query(jpegs)
    n = len(jpegs)
    stage_host = torch.zeros(sz.stage_bytes, dtype=torch.uint8).pin_memory()
    stage_dev = torch.zeros(sz.stage_bytes, dtype=torch.uint8, device=dev)
    coef = torch.full((max(1, sz.coef_bytes // 2),), 77, dtype=torch.int16, device=dev)
    pix_buf = torch.full((GUARD + sz.packed_bytes + GUARD,), CANARY, dtype=torch.uint8, device=dev)
    pixels = pix_buf[GUARD:GUARD + sz.packed_bytes]
    table = torch.zeros(16 * n, dtype=torch.uint8, device=dev)
    table_host = torch.zeros(16 * n, dtype=torch.uint8).pin_memory()
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    call = pb.PreparedJpeg(jpegs, stage_host, stage_dev, coef, pixels, table, table_host, status)
    call()
    torch.cuda.synchronize()
    assert int(status.item()) == expect_status, pb.preba_strerror(int(status.item()))
    host = pix_buf.cpu().numpy()
    assert np.all(host[:GUARD] == CANARY) and np.all(host[GUARD + sz.packed_bytes:] == CANARY), \
        "kernel wrote outside the pixel buffer"
    packed = host[GUARD:GUARD + sz.packed_bytes]
    tab = table.cpu().numpy().view(pb.TABLE_DTYPE)
    assert np.array_equal(tab, table_host.numpy().view(pb.TABLE_DTYPE))
    images, at = [], 0
    for i in range(n):
        assert (int(tab[i]["offset"]), int(tab[i]["h"]), int(tab[i]["w"])) == (at, int(h[i]), int(w[i]))
        nb = 3 * int(h[i]) * int(w[i])
        images.append(packed[at:at + nb].reshape(int(h[i]), int(w[i]), 3).copy())
        at = -(-(at + nb) // 128) * 128
    return images, coef.cpu().numpy(), (pixels, table, sz)


def device_order(planes, frame):
    """The oracle's coefficient planes in the order the device stores them: MCU after MCU, in
    each the blocks of component 0, 1, 2, raster order inside the MCU."""
    rows, cols = frame.mcus
    out = []
    for my in range(rows):
        for mx in range(cols):
            for c, p in zip(frame.components, planes):
                for by in range(c["v"]):
                    for bx in range(c["h"]):
                        out.append(p[my * c["v"] + by, mx * c["h"] + bx])
    return np.asarray(out, dtype=np.int32).reshape(-1)


def synthetic(seed, h, w):
    return wl.smooth_image(np.random.default_rng(seed), h, w, jitter=24.0)


@pytest.mark.gpu
@pytest.mark.parametrize("subsampling,restart_rows", [(0, 0), (0, 1), (1, 1), (2, 0), (2, 1), (2, 3)])
def test_ragged_batch_bit_for_bit(subsampling, restart_rows):
    sizes = [(40, 50), (75, 101), (33, 9), (8, 8), (1, 1), (17, 160), (250, 333)]
    imgs = [synthetic(10 * subsampling + i, h, w) for i, (h, w) in enumerate(sizes)]
    jpegs = wl.jpeg_streams(imgs, quality=88, subsampling=subsampling, restart_rows=restart_rows)
    got, coef, _ = decode_on_gpu(jpegs)
    at = 0
    for j, g in zip(jpegs, got):
        f = oj.parse(j)
        want_coef = device_order(oj.entropy_decode(j, f), f)
        assert np.array_equal(coef[at:at + want_coef.size].astype(np.int32), want_coef)
        at += want_coef.size
        assert np.array_equal(g, oj.decode(j))


@pytest.mark.gpu
def test_grey_streams_qualities_and_noise():
    from PIL import Image

    jpegs = []
    for k, q in enumerate((30, 75, 100)):
        buf = io.BytesIO()
        Image.fromarray(synthetic(40 + k, 61, 77)[:, :, 0]).save(buf, format="JPEG", quality=q)
        jpegs.append(buf.getvalue())
    jpegs += wl.jpeg_streams([synthetic(50, 64, 64)], quality=100, subsampling=0, restart_rows=0)
    # uniform noise: long codes, large coefficients, many escapes of 0xFF
    noise = wl.uniform_image(np.random.default_rng(51), 48, 80)
    jpegs += wl.jpeg_streams([noise], quality=100, subsampling=2, restart_rows=1)
    got, _, _ = decode_on_gpu(jpegs)
    for j, g in zip(jpegs, got):
        assert np.array_equal(g, oj.decode(j))


@pytest.mark.gpu
def test_decode_feeds_the_transform():
    """Decode, then preba_preprocess on the buffers Decode wrote, on the same stream."""
    import torch

    imgs = wl.mixed_smooth(6, seed=71)
    jpegs = wl.jpeg_streams(imgs, quality=90, subsampling=2, restart_rows=1)
    decoded, _, (pixels, table, sz) = decode_on_gpu(jpegs)
    n = len(jpegs)
    dev = torch.device("cuda:0")
    out = torch.empty((n, 3, 224, 224), dtype=torch.float32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    pb.preba_preprocess(pixels, table, n, out, 224, 256, MEAN, STD, pb.F32, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    want_imgs = [oj.decode(j) for j in jpegs]
    for d, wimg in zip(decoded, want_imgs):
        assert np.array_equal(d, wimg)
    want = oracle.preprocess(want_imgs, 224, 256, MEAN, STD, oracle.OUT_F64, nthreads=host_threads())
    assert float(np.max(np.abs(out.cpu().numpy().astype(np.float64) - want))) <= FP32_TOL


@pytest.mark.gpu
def test_full_size_images_sampled():
    imgs = wl.mixed_smooth(12, seed=72)
    jpegs = wl.jpeg_streams(imgs, quality=90, subsampling=2, restart_rows=1)
    got, _, _ = decode_on_gpu(jpegs)
    for k in (0, 5, 11):                         # the oracle takes seconds per image
        assert np.array_equal(got[k], oj.decode(jpegs[k]))
    for g, im in zip(got, imgs):                 # and every image is its source, within the loss
        assert float(np.mean(np.abs(g.astype(int) - im.astype(int)))) <= 6.0


@pytest.mark.gpu
def test_damaged_stream_is_reported_not_followed():
    imgs = [synthetic(80, 64, 96), synthetic(81, 40, 40)]
    jpegs = wl.jpeg_streams(imgs, quality=85, subsampling=2, restart_rows=1)
    f = oj.parse(jpegs[0])
    broken = bytearray(jpegs[0])
    k = broken.index(b"\xff\xd1", f.scan_start)   # drop one restart marker: the count is off
    del broken[k:k + 2]
    got, _, _ = decode_on_gpu([bytes(broken), jpegs[1]], expect_status=pb.ERR_BAD_STREAM)
    assert np.array_equal(got[1], oj.decode(jpegs[1]))   # the neighbour is untouched by it


@pytest.mark.parametrize("case", ["progressive", "cmyk", "truncated", "not-jpeg", "twelve-bit"])
def test_refusals_before_any_launch(case):
    from PIL import Image

    img = synthetic(90, 40, 40)
    buf = io.BytesIO()
    if case == "progressive":
        Image.fromarray(img).save(buf, format="JPEG", progressive=True)
        data, want = buf.getvalue(), pb.ERR_UNSUPPORTED
    elif case == "cmyk":
        Image.fromarray(np.dstack([img, img[:, :, :1]]), mode="CMYK").save(buf, format="JPEG")
        data, want = buf.getvalue(), pb.ERR_UNSUPPORTED
    elif case == "truncated":
        Image.fromarray(img).save(buf, format="JPEG")
        data, want = buf.getvalue()[:120], pb.ERR_BAD_STREAM
    elif case == "twelve-bit":
        Image.fromarray(img).save(buf, format="JPEG")
        data = bytearray(buf.getvalue())
        data[data.index(b"\xff\xc0") + 4] = 12
        data, want = bytes(data), pb.ERR_UNSUPPORTED
    else:
        data, want = b"\x89PNG\r\n\x1a\n" + bytes(64), pb.ERR_BAD_STREAM
    with pytest.raises(pb.PrebaError) as e:
        pb.preba_jpeg_query([data])
    assert e.value.code == want
    with pytest.raises((oj.Unsupported, ValueError)):
        oj.decode(data)
