"""Host side of the C ABI: exported symbols, sizes, packing (bit-exact), error codes.
No call here reaches the device."""
from __future__ import annotations

import ctypes
import re
from pathlib import Path

import numpy as np
import pytest

import oracle
from paper_2411_19114_b200 import binding as pb
from paper_2411_19114_b200 import build as pbuild

ROOT = Path(__file__).resolve().parent.parent
MEAN = (0.485, 0.456, 0.406)
STD = (0.229, 0.224, 0.225)


@pytest.fixture(scope="module", autouse=True)
def built_library():
    pbuild.build()


def declared_functions() -> list[str]:
    names = []
    for header in sorted((ROOT / "include").glob("*.h")):
        text = re.sub(r"/\*.*?\*/", "", header.read_text(), flags=re.S)
        names += re.findall(r"\b(preba_[a-z_0-9]+)\s*\(", text)
    return sorted(set(names))


def test_library_exports_every_declared_function():
    names = declared_functions()
    assert set(names) == set(pb.EXPORTS)
    handle = ctypes.CDLL(str(pbuild.LIB))
    for name in names:
        assert getattr(handle, name) is not None


def test_header_is_plain_c(tmp_path):
    """include/preba.h promises plain C: it must compile as C11 on its own, and the struct
    sizes the binding assumes must be the compiler's."""
    import subprocess

    src = tmp_path / "use_header.c"
    src.write_text(
        '#include "preba.h"\n#include <stdio.h>\n'
        "int main(void) { printf(\"%zu %zu %zu %zu %zu %zu %zu %zu %zu %zu\\n\", sizeof(preba_img_t), "
        "sizeof(preba_sizes_t), sizeof(preba_batch_t), sizeof(preba_host_batch_t), "
        "sizeof(preba_image_batch_t), sizeof(preba_options_t), sizeof(preba_utt_t), "
        "sizeof(preba_audio_sizes_t), sizeof(preba_audio_batch_t), sizeof(preba_serve_t)); "
        "printf(\"%zu %zu\\n\", sizeof(preba_jpeg_sizes_t), sizeof(preba_jpeg_batch_t)); "
        "return 0; }\n")
    exe = tmp_path / "use_header"
    subprocess.run(["gcc", "-std=c11", "-Wall", "-Wextra", "-Werror", "-pedantic",
                    "-I", str(ROOT / "include"), "-o", str(exe), str(src)], check=True)
    sizes = [int(v) for v in subprocess.run([str(exe)], check=True, capture_output=True,
                                            text=True).stdout.split()]
    assert sizes == [ctypes.sizeof(pb.PrebaImg), ctypes.sizeof(pb.PrebaSizes),
                     ctypes.sizeof(pb.PrebaBatch), ctypes.sizeof(pb.PrebaHostBatch),
                     ctypes.sizeof(pb.PrebaImageBatch), ctypes.sizeof(pb.PrebaOptions),
                     pb.UTT_DTYPE.itemsize, ctypes.sizeof(pb.PrebaAudioSizes),
                     ctypes.sizeof(pb.PrebaAudioBatch), ctypes.sizeof(pb.PrebaServe),
                     ctypes.sizeof(pb.PrebaJpegSizes), ctypes.sizeof(pb.PrebaJpegBatch)]


def test_struct_layouts_match_header():
    assert ctypes.sizeof(pb.PrebaImg) == 16 and pb.TABLE_DTYPE.itemsize == 16
    assert ctypes.sizeof(pb.PrebaSizes) == 32
    assert ctypes.sizeof(pb.PrebaBatch) == 72
    assert ctypes.sizeof(pb.PrebaHostBatch) == 88
    assert ctypes.sizeof(pb.PrebaImageBatch) == 104


def test_query_sizes():
    h, w = [240, 1, 375, 17], [320, 1, 500, 43]
    s = pb.preba_query(h, w, 224, pb.F16)
    at = 0
    for hh, ww in zip(h, w):
        at = -(-(at + 3 * hh * ww) // 128) * 128
    assert s.packed_bytes == at and s.align == 128
    assert s.table_bytes == 16 * 4
    assert s.out_bytes == 4 * 3 * 224 * 224 * 2
    assert pb.preba_query(h, w, 224, pb.F32).out_bytes == 4 * 3 * 224 * 224 * 4
    assert pb.preba_query(h, w, 224, pb.BF16).out_bytes == 4 * 3 * 224 * 224 * 2
    # largest accepted image: no overflow
    s = pb.preba_query([32768, 32768], [32768, 32768], 1, pb.F32)
    assert s.packed_bytes == 2 * 3 * 32768 * 32768


@pytest.mark.parametrize("h,w,c,dt", [([0], [5], 8, 0), ([5], [0], 8, 0), ([32769], [5], 8, 0),
                                      ([5], [5], 0, 0), ([5], [5], 8, 3), ([5], [5], 8, -1),
                                      ([], [], 8, 0)])
def test_query_rejects(h, w, c, dt):
    with pytest.raises(pb.PrebaError) as e:
        pb.preba_query(h, w, c, dt)
    assert e.value.code == pb.ERR_INVALID_ARG


@pytest.mark.parametrize("seed", range(4))
def test_pack_is_bit_exact_against_oracle(seed):
    rng = np.random.default_rng(200 + seed)
    n = int(rng.integers(1, 12))
    imgs = [rng.integers(0, 256, size=(int(rng.integers(1, 70)), int(rng.integers(1, 70)), 3),
                         dtype=np.uint8) for _ in range(n)]
    want_packed, want_off, want_h, want_w = oracle.pack(imgs)
    total = pb.preba_query(want_h, want_w, 1, pb.F32).packed_bytes
    assert total == len(want_packed)
    packed = np.full(total + 256, 0xA5, dtype=np.uint8)  # guard band behind the buffer
    table = np.zeros(n, dtype=pb.TABLE_DTYPE)
    pb.preba_pack(imgs, packed[:total], table)
    assert np.array_equal(packed[:total], want_packed)
    assert np.all(packed[total:] == 0xA5)
    assert np.array_equal(table["offset"], want_off)
    assert np.array_equal(table["h"], want_h) and np.array_equal(table["w"], want_w)
    # idempotent: packing again over the old contents gives the same bytes
    pb.preba_pack(imgs, packed[:total], table)
    assert np.array_equal(packed[:total], want_packed)


def test_pack_errors():
    img = np.zeros((4, 4, 3), dtype=np.uint8)
    with pytest.raises(pb.PrebaError) as e:
        pb.preba_pack([img], np.zeros(127, dtype=np.uint8))
    assert e.value.code == pb.ERR_BUFFER_TOO_SMALL
    L = pb.lib()
    h = (ctypes.c_uint32 * 1)(4)
    w = (ctypes.c_uint32 * 1)(4)
    buf = np.zeros(128, dtype=np.uint8)
    tab = np.zeros(1, dtype=pb.TABLE_DTYPE)
    ptrs = (ctypes.c_void_p * 1)(None)
    assert L.preba_pack(ptrs, h, w, 1, buf.ctypes.data, 128, tab.ctypes.data) == pb.ERR_INVALID_ARG
    assert L.preba_pack(None, h, w, 1, buf.ctypes.data, 128, tab.ctypes.data) == pb.ERR_INVALID_ARG
    ptrs = (ctypes.c_void_p * 1)(img.ctypes.data)
    assert L.preba_pack(ptrs, h, w, 0, buf.ctypes.data, 128, tab.ctypes.data) == pb.ERR_INVALID_ARG
    assert L.preba_pack(ptrs, h, w, 1, None, 128, tab.ctypes.data) == pb.ERR_INVALID_ARG
    assert L.preba_pack(ptrs, h, w, 1, buf.ctypes.data, 128, None) == pb.ERR_INVALID_ARG


def test_strerror_covers_every_code():
    texts = {pb.preba_strerror(c) for c in range(0, -11, -1)}
    assert len(texts) == 11 and "ok" in texts
    assert "unknown" in pb.preba_strerror(-99)


def _batch(**kw):
    """A batch with plausible (fake, never dereferenced) device addresses."""
    b = pb.PrebaBatch()
    b.pixels, b.pixels_bytes = 0x10000, 1 << 20
    b.table, b.table_host = 0x20000, None
    b.n = 2
    b.out, b.out_bytes = 0x30000, 2 * 3 * 16 * 16 * 4
    b.status = None
    for k, v in kw.items():
        setattr(b, k, v)
    return b


def _call(batch, c=16, s=16, mean=MEAN, std=STD, dt=pb.F32):
    m = (ctypes.c_float * 3)(*mean)
    sd = (ctypes.c_float * 3)(*std)
    return pb.lib().preba_preprocess(ctypes.byref(batch) if batch is not None else None, c, s,
                                     m, sd, dt, None)


def test_preprocess_rejects_bad_arguments_before_any_launch():
    assert _call(None) == pb.ERR_INVALID_ARG
    assert _call(_batch(pixels=None)) == pb.ERR_INVALID_ARG
    assert _call(_batch(table=None)) == pb.ERR_INVALID_ARG
    assert _call(_batch(out=None)) == pb.ERR_INVALID_ARG
    assert _call(_batch(n=0)) == pb.ERR_INVALID_ARG
    assert _call(_batch(pixels=0x10001)) == pb.ERR_INVALID_ARG      # misaligned pixels
    assert _call(_batch(out=0x30008)) == pb.ERR_INVALID_ARG         # misaligned out
    assert _call(_batch(scratch=0x40004)) == pb.ERR_INVALID_ARG     # misaligned scratch
    assert _call(_batch(flags=2)) == pb.ERR_INVALID_ARG             # unknown flag
    assert _call(_batch(), c=0) == pb.ERR_INVALID_ARG
    assert _call(_batch(), c=17, s=16) == pb.ERR_INVALID_ARG        # crop larger than resize
    assert _call(_batch(), s=16385) == pb.ERR_INVALID_ARG
    assert _call(_batch(), dt=3) == pb.ERR_INVALID_ARG
    assert _call(_batch(), std=(0.2, 0.0, 0.2)) == pb.ERR_INVALID_ARG
    assert _call(_batch(), std=(0.2, float("inf"), 0.2)) == pb.ERR_INVALID_ARG
    assert _call(_batch(), mean=(float("nan"), 0.1, 0.2)) == pb.ERR_INVALID_ARG
    assert _call(_batch(out_bytes=2 * 3 * 16 * 16 * 4 - 1)) == pb.ERR_BUFFER_TOO_SMALL
    assert _call(_batch(pixels_bytes=0)) == pb.ERR_BUFFER_TOO_SMALL


def test_preprocess_checks_host_table_before_launch():
    def table(entries):
        t = np.zeros(len(entries), dtype=pb.TABLE_DTYPE)
        for i, e in enumerate(entries):
            t[i] = e
        return t

    for bad in ([(0, 8, 8), (64, 8, 8)],            # misaligned offset
                [(0, 8, 8), (128, 0, 8)],           # zero height
                [(0, 8, 8), (128, 8, 40000)],       # width out of range
                [(0, 8, 8), ((1 << 20) - 128, 8, 8)],  # runs past the pixel buffer
                [(0, 8, 8), (1 << 40, 8, 8)]):      # offset past the pixel buffer
        t = table(bad)
        assert _call(_batch(table_host=t.ctypes.data)) == pb.ERR_BAD_TABLE


def test_extended_entry_point_rejects_bad_arguments_before_any_launch():
    def call(batch=None, **kw):
        b = batch if batch is not None else _batch(out_bytes=2 * 3 * 16 * 16 * 4)
        o = pb.PrebaOptions()
        o.out_size, o.resize_short = 16, 16
        o.mean = (ctypes.c_float * 3)(*MEAN)
        o.std = (ctypes.c_float * 3)(*STD)
        o.out_dtype, o.flags = pb.F32, 0
        for k, v in kw.items():
            setattr(o, k, v)
        return pb.lib().preba_preprocess_ex(ctypes.byref(b), ctypes.byref(o), None)

    assert pb.lib().preba_preprocess_ex(None, None, None) == pb.ERR_INVALID_ARG
    assert call(flags=2) == pb.ERR_INVALID_ARG                       # unknown flag
    assert call(out_dtype=pb.U8) == pb.ERR_INVALID_ARG               # uint8 output needs rounding
    assert call(out_dtype=4, flags=pb.EX_ROUND_U8) == pb.ERR_INVALID_ARG
    assert call(out_size=17) == pb.ERR_INVALID_ARG
    assert call(crop_origin=0x50002) == pb.ERR_INVALID_ARG           # misaligned table of windows
    assert call(std=(ctypes.c_float * 3)(0.2, 0.0, 0.2)) == pb.ERR_INVALID_ARG
    assert call(_batch(out_bytes=2 * 16 * 16 * 3 - 1), out_dtype=pb.U8,
                flags=pb.EX_ROUND_U8) == pb.ERR_BUFFER_TOO_SMALL     # one byte per element
    # windows checked on the host when both host copies are there: S = 16, C = 16
    t = np.zeros(2, dtype=pb.TABLE_DTYPE)
    t[0], t[1] = (0, 8, 8), (256, 8, 16)                             # resized 16 x 16 and 16 x 32
    bad = np.asarray([0, 0, 0, 17], dtype=np.uint32)                 # 17 + 16 > 32
    b = _batch(out_bytes=2 * 3 * 16 * 16 * 4, table_host=t.ctypes.data)
    assert call(b, crop_origin=0x50000, crop_origin_host=bad.ctypes.data) == pb.ERR_BAD_CROP
    assert pb.preba_strerror(pb.ERR_BAD_CROP) != pb.preba_strerror(-99)


def test_antialiased_entry_point_rejects_bad_arguments_before_any_launch():
    def call(batch=None, **kw):
        b = batch if batch is not None else _batch(out_bytes=2 * 3 * 16 * 16 * 4)
        o = pb.PrebaOptions()
        o.out_size, o.resize_short = 16, 16
        o.mean = (ctypes.c_float * 3)(*MEAN)
        o.std = (ctypes.c_float * 3)(*STD)
        o.out_dtype, o.flags = pb.F32, 0
        for k, v in kw.items():
            setattr(o, k, v)
        return pb.lib().preba_preprocess_antialias(ctypes.byref(b), ctypes.byref(o), None)

    assert pb.lib().preba_preprocess_antialias(None, None, None) == pb.ERR_INVALID_ARG
    assert call(flags=pb.EX_ROUND_U8) == pb.ERR_INVALID_ARG          # no rounding in this variant
    assert call(out_dtype=pb.U8) == pb.ERR_INVALID_ARG
    assert call(out_size=17) == pb.ERR_INVALID_ARG                   # crop larger than the resize
    assert call(out_size=0) == pb.ERR_INVALID_ARG
    assert call(resize_short=16384 + 1, out_size=16) == pb.ERR_INVALID_ARG   # PREBA_MAX_RESIZE
    assert call(crop_origin=0x50002) == pb.ERR_INVALID_ARG           # misaligned table of windows
    assert call(std=(ctypes.c_float * 3)(0.2, 0.0, 0.2)) == pb.ERR_INVALID_ARG
    assert call(mean=(ctypes.c_float * 3)(0.2, float("nan"), 0.2)) == pb.ERR_INVALID_ARG
    assert call(_batch(out_bytes=2 * 3 * 16 * 16 * 4 - 1)) == pb.ERR_BUFFER_TOO_SMALL


def test_separate_images_entry_point_rejects_bad_arguments_before_any_copy():
    """preba_preprocess_images validates on the host first: nothing below reaches CUDA."""
    img = np.zeros((8, 8, 3), dtype=np.uint8)
    ptrs = (ctypes.c_void_p * 2)(img.ctypes.data, img.ctypes.data)
    h = np.array([8, 8], dtype=np.uint32)
    w = np.array([8, 8], dtype=np.uint32)
    tab = np.zeros(2, dtype=pb.TABLE_DTYPE)

    def call(c=8, s=8, **kw):
        b = pb.PrebaImageBatch()
        b.images = ctypes.cast(ptrs, ctypes.c_void_p)
        b.h, b.w, b.n = h.ctypes.data, w.ctypes.data, 2
        b.table_host = tab.ctypes.data
        b.out_host, b.out_bytes = 0x50000, 2 * 3 * 8 * 8 * 4
        b.dev_pixels, b.dev_pixels_bytes = 0x10000, 512
        b.dev_table, b.dev_out = 0x20000, 0x30000
        for k, v in kw.items():
            setattr(b, k, v)
        m = (ctypes.c_float * 3)(*MEAN)
        sd = (ctypes.c_float * 3)(*STD)
        return pb.lib().preba_preprocess_images(ctypes.byref(b), c, s, m, sd, pb.F32, None)

    assert pb.lib().preba_preprocess_images(None, 8, 8, None, None, pb.F32, None) == pb.ERR_INVALID_ARG
    assert call(images=None) == pb.ERR_INVALID_ARG
    assert call(table_host=None) == pb.ERR_INVALID_ARG
    assert call(out_host=None) == pb.ERR_INVALID_ARG
    assert call(dev_table=None) == pb.ERR_INVALID_ARG
    assert call(n=0) == pb.ERR_INVALID_ARG
    assert call(dev_pixels_bytes=511) == pb.ERR_BUFFER_TOO_SMALL   # two images of 192 -> 256 bytes each
    assert call(out_bytes=2 * 3 * 8 * 8 * 4 - 1) == pb.ERR_BUFFER_TOO_SMALL
    assert call(dev_pixels=0x10004) == pb.ERR_INVALID_ARG          # misaligned staging
    assert call(c=9, s=8) == pb.ERR_INVALID_ARG                    # crop larger than resize
    assert call(flags=4) == pb.ERR_INVALID_ARG                     # unknown flag
    raw = np.zeros(8 * 8 * 3 + 256, dtype=np.uint8)
    odd = raw.ctypes.data + (64 - raw.ctypes.data) % 128           # an address that is 64 mod 128
    assert odd % 128 == 64
    two = (ctypes.c_void_p * 2)(odd, odd)
    assert call(flags=pb.IMAGES_IN_PLACE, images=ctypes.cast(two, ctypes.c_void_p)) \
        == pb.ERR_INVALID_ARG                                      # in place wants 128-byte aligned images
    # the table is written before the checks that follow it: the layout of preba_pack
    assert [int(e["offset"]) for e in tab] == [0, 256]
    w[1] = 0
    assert call() == pb.ERR_INVALID_ARG                            # zero width


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(pb, "_lib", None)
    monkeypatch.setattr(pb, "_LIB_PATH", tmp_path / "libpreba.so")
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        pb.lib()
