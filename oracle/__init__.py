"""TEST INFRASTRUCTURE ONLY: Python access to the CPU oracle in ``preba_oracle.c``.

The oracle is the plain double-precision definition of the preprocessing path
(resize -> center crop -> normalise -> HWC->NCHW; paper Sec. 2.3 item 1, Fig. 4,
Table 1).  Only the tests, the smoke check and the benchmark's CPU-baseline leg
may import this package.  It shares nothing with the CUDA library: its C source
is compiled here with gcc into ``liboracle.so`` and called through ctypes; this
module only marshals arguments.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "preba_oracle.c"
_SRC_VARIANTS = _HERE / "preba_oracle_variants.c"
_LIB = _HERE / "liboracle.so"

PACK_ALIGN = 128
OUT_F64, OUT_F32, OUT_F16, OUT_BF16, OUT_U8_HWC = 0, 1, 2, 3, 4

_lib = None


def build(force: bool = False) -> Path:
    """Compile the oracle (gcc -O2, no fast-math) if the library is missing or stale."""
    newest = max(_SRC.stat().st_mtime, _SRC_VARIANTS.stat().st_mtime)
    if force or not _LIB.exists() or _LIB.stat().st_mtime < newest:
        tmp = _LIB.with_suffix(f".tmp{os.getpid()}.so")
        subprocess.run(
            ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-Wall", "-Wextra",
             "-o", str(tmp), str(_SRC), str(_SRC_VARIANTS), "-lm", "-lpthread"],
            check=True,
        )
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(str(_LIB))
        u8p = ctypes.POINTER(ctypes.c_uint8)
        u32p = ctypes.POINTER(ctypes.c_uint32)
        u64p = ctypes.POINTER(ctypes.c_uint64)
        f32p = ctypes.POINTER(ctypes.c_float)
        f64p = ctypes.POINTER(ctypes.c_double)
        lib.oracle_resized_size.argtypes = [ctypes.c_uint32] * 3 + [u64p, u64p]
        lib.oracle_axis.argtypes = [ctypes.c_uint32, ctypes.c_uint64, ctypes.c_uint32,
                                    ctypes.c_uint32, u32p, u32p, f64p]
        lib.oracle_element.argtypes = [u8p, ctypes.c_uint32, ctypes.c_uint32, ctypes.c_uint32,
                                       ctypes.c_uint32, f32p, f32p, ctypes.c_uint32,
                                       ctypes.c_uint32, ctypes.c_uint32, f64p]
        lib.oracle_round_f16.argtypes = [ctypes.c_double]
        lib.oracle_round_f16.restype = ctypes.c_uint16
        lib.oracle_round_bf16.argtypes = [ctypes.c_double]
        lib.oracle_round_bf16.restype = ctypes.c_uint16
        lib.oracle_pack_size.argtypes = [u32p, u32p, ctypes.c_uint32, u64p]
        lib.oracle_pack.argtypes = [ctypes.POINTER(u8p), u32p, u32p, ctypes.c_uint32, u8p,
                                    ctypes.c_uint64, u64p]
        lib.oracle_preprocess.argtypes = [u8p, u64p, u32p, u32p, ctypes.c_uint32,
                                          ctypes.c_uint32, ctypes.c_uint32, f32p, f32p,
                                          ctypes.c_int, ctypes.c_void_p, ctypes.c_uint32]
        lib.oracle_var_axis.argtypes = [ctypes.c_uint32, ctypes.c_uint64, ctypes.c_uint64,
                                        ctypes.c_uint32, u32p, u32p, u64p, u64p]
        lib.oracle_var_value.argtypes = [u8p, ctypes.c_uint32, ctypes.c_uint32, ctypes.c_uint32,
                                         ctypes.c_uint32, ctypes.c_uint64, ctypes.c_uint64,
                                         ctypes.c_uint32, ctypes.c_uint32, ctypes.c_uint32, f64p]
        lib.oracle_var_pixel_u8.argtypes = [u8p, ctypes.c_uint32, ctypes.c_uint32, ctypes.c_uint32,
                                            ctypes.c_uint32, ctypes.c_uint64, ctypes.c_uint64,
                                            ctypes.c_uint32, ctypes.c_uint32, ctypes.c_uint32, u8p]
        lib.oracle_var_preprocess.argtypes = [u8p, u64p, u32p, u32p, ctypes.c_uint32,
                                              ctypes.c_uint32, ctypes.c_uint32, f32p, f32p, u32p,
                                              ctypes.c_int, ctypes.c_int, ctypes.c_void_p,
                                              ctypes.c_uint32]
        _lib = lib
    return _lib


def _ptr(a: np.ndarray, ctype):
    return a.ctypes.data_as(ctypes.POINTER(ctype))


def _f3(v) -> np.ndarray:
    a = np.ascontiguousarray(np.asarray(v, dtype=np.float32))
    if a.shape != (3,):
        raise ValueError("mean/std must have 3 entries")
    return a


def _check(rc: int, what: str) -> None:
    if rc != 0:
        raise ValueError(f"{what}: oracle error {rc}")


def resized_size(h: int, w: int, s: int) -> tuple[int, int]:
    """(R_h, R_w): shorter side -> s, longer -> floor(s*long/short)."""
    rh, rw = ctypes.c_uint64(), ctypes.c_uint64()
    _check(_load().oracle_resized_size(h, w, s, ctypes.byref(rh), ctypes.byref(rw)), "resized_size")
    return rh.value, rw.value


def axis(n_in: int, r: int, c: int, j: int) -> tuple[int, int, float]:
    """Taps (i0, i1) and weight of i1 for crop-window index j along one axis."""
    i0, i1, lam = ctypes.c_uint32(), ctypes.c_uint32(), ctypes.c_double()
    _check(_load().oracle_axis(n_in, r, c, j, ctypes.byref(i0), ctypes.byref(i1),
                               ctypes.byref(lam)), "axis")
    return i0.value, i1.value, lam.value


def element(img: np.ndarray, c: int, s: int, mean, std, ch: int, k: int, j: int) -> float:
    """out[ch, k, j] of one HWC uint8 image, in double."""
    img = np.ascontiguousarray(img, dtype=np.uint8)
    h, w, three = img.shape
    assert three == 3
    m, sd = _f3(mean), _f3(std)
    out = ctypes.c_double()
    _check(_load().oracle_element(_ptr(img, ctypes.c_uint8), h, w, c, s,
                                  _ptr(m, ctypes.c_float), _ptr(sd, ctypes.c_float),
                                  ch, k, j, ctypes.byref(out)), "element")
    return out.value


def round_f16_bits(x: float) -> int:
    """binary16 bit pattern of x rounded once, ties to even."""
    return int(_load().oracle_round_f16(float(x)))


def round_bf16_bits(x: float) -> int:
    """bfloat16 bit pattern of x rounded once, ties to even."""
    return int(_load().oracle_round_bf16(float(x)))


def pack(images: list[np.ndarray]) -> tuple[np.ndarray, np.ndarray, np.ndarray, np.ndarray]:
    """Packed byte buffer, offsets (uint64), h, w (uint32) of a list of HWC uint8 images."""
    imgs = [np.ascontiguousarray(im, dtype=np.uint8) for im in images]
    n = len(imgs)
    h = np.array([im.shape[0] for im in imgs], dtype=np.uint32)
    w = np.array([im.shape[1] for im in imgs], dtype=np.uint32)
    total = ctypes.c_uint64()
    lib = _load()
    _check(lib.oracle_pack_size(_ptr(h, ctypes.c_uint32), _ptr(w, ctypes.c_uint32), n,
                                ctypes.byref(total)), "pack_size")
    packed = np.full(total.value, 0xEE, dtype=np.uint8)  # poison: pack must write every byte
    offsets = np.zeros(n, dtype=np.uint64)
    u8p = ctypes.POINTER(ctypes.c_uint8)
    ptrs = (u8p * n)(*[_ptr(im, ctypes.c_uint8) for im in imgs])
    _check(lib.oracle_pack(ptrs, _ptr(h, ctypes.c_uint32), _ptr(w, ctypes.c_uint32), n,
                           _ptr(packed, ctypes.c_uint8), total.value,
                           _ptr(offsets, ctypes.c_uint64)), "pack")
    return packed, offsets, h, w


def preprocess_packed(packed: np.ndarray, offsets: np.ndarray, h: np.ndarray, w: np.ndarray,
                      c: int, s: int, mean, std, out_kind: int = OUT_F64,
                      nthreads: int = 1) -> np.ndarray:
    """[n,3,c,c] result for a packed batch; float64, float32, float16, or bfloat16 as uint16
    bit patterns (one rounding each)."""
    packed = np.ascontiguousarray(packed, dtype=np.uint8)
    offsets = np.ascontiguousarray(offsets, dtype=np.uint64)
    h = np.ascontiguousarray(h, dtype=np.uint32)
    w = np.ascontiguousarray(w, dtype=np.uint32)
    n = len(h)
    dt = {OUT_F64: np.float64, OUT_F32: np.float32, OUT_F16: np.uint16, OUT_BF16: np.uint16}[out_kind]
    out = np.empty((n, 3, c, c), dtype=dt)
    m, sd = _f3(mean), _f3(std)
    _check(_load().oracle_preprocess(_ptr(packed, ctypes.c_uint8), _ptr(offsets, ctypes.c_uint64),
                                     _ptr(h, ctypes.c_uint32), _ptr(w, ctypes.c_uint32), n, c, s,
                                     _ptr(m, ctypes.c_float), _ptr(sd, ctypes.c_float),
                                     out_kind, out.ctypes.data_as(ctypes.c_void_p), nthreads),
           "preprocess")
    return out.view(np.float16) if out_kind == OUT_F16 else out


def preprocess(images: list[np.ndarray], c: int, s: int, mean, std, out_kind: int = OUT_F64,
               nthreads: int = 1) -> np.ndarray:
    """Pack a list of HWC uint8 images and run the oracle over the batch."""
    packed, offsets, h, w = pack(images)
    return preprocess_packed(packed, offsets, h, w, c, s, mean, std, out_kind, nthreads)


# ---- variants: explicit crop origins, rounding to uint8 (preba_oracle_variants.c) ---------------

def var_axis(n_in: int, r: int, origin: int, j: int) -> tuple[int, int, int, int]:
    """Taps (i0, i1), remainder and denominator for resized index origin + j along one axis."""
    i0, i1 = ctypes.c_uint32(), ctypes.c_uint32()
    rem, den = ctypes.c_uint64(), ctypes.c_uint64()
    _check(_load().oracle_var_axis(n_in, r, origin, j, ctypes.byref(i0), ctypes.byref(i1),
                                   ctypes.byref(rem), ctypes.byref(den)), "var_axis")
    return i0.value, i1.value, rem.value, den.value


def var_pixel_u8(img: np.ndarray, c: int, s: int, top: int, left: int, ch: int, k: int,
                 j: int) -> int:
    """Rounded (ties up) bilinear pixel of one HWC uint8 image for a window at (top, left)."""
    img = np.ascontiguousarray(img, dtype=np.uint8)
    h, w, _ = img.shape
    q = ctypes.c_uint8()
    _check(_load().oracle_var_pixel_u8(_ptr(img, ctypes.c_uint8), h, w, c, s, top, left, ch, k, j,
                                       ctypes.byref(q)), "var_pixel_u8")
    return q.value


def preprocess_ex(images: list[np.ndarray], c: int, s: int, mean, std, out_kind: int = OUT_F64,
                  crop_origin=None, round_u8: bool = False, nthreads: int = 1) -> np.ndarray:
    """The batch with an explicit crop origin per image (``crop_origin``: n pairs (top, left)
    on the resized grid, None = centre) and/or rounding of the resized pixel to uint8.
    Float kinds give [n,3,c,c]; OUT_U8_HWC gives the rounded pixels as [n,c,c,3] uint8."""
    packed, offsets, h, w = pack(images)
    n = len(images)
    if out_kind == OUT_U8_HWC:
        out = np.empty((n, c, c, 3), dtype=np.uint8)
    else:
        dt = {OUT_F64: np.float64, OUT_F32: np.float32, OUT_F16: np.uint16,
              OUT_BF16: np.uint16}[out_kind]
        out = np.empty((n, 3, c, c), dtype=dt)
    m, sd = _f3(mean), _f3(std)
    co = None
    if crop_origin is not None:
        co = np.ascontiguousarray(np.asarray(crop_origin, dtype=np.uint32).reshape(n, 2))
    _check(_load().oracle_var_preprocess(
        _ptr(packed, ctypes.c_uint8), _ptr(offsets, ctypes.c_uint64), _ptr(h, ctypes.c_uint32),
        _ptr(w, ctypes.c_uint32), n, c, s, _ptr(m, ctypes.c_float), _ptr(sd, ctypes.c_float),
        _ptr(co, ctypes.c_uint32) if co is not None else None, int(round_u8), out_kind,
        out.ctypes.data_as(ctypes.c_void_p), nthreads), "preprocess_ex")
    return out.view(np.float16) if out_kind == OUT_F16 else out
