"""ctypes binding of ``libpreba.so`` — argument marshalling only.

Function names and meanings are those of ``include/preba.h``.  Device memory and
streams come from PyTorch; nothing here computes any part of the transform.  If
the library has not been built the first call raises: there is no fallback.
"""
from __future__ import annotations

import ctypes
import os
from pathlib import Path

import numpy as np

# PREBA_CHECKED_BUILD=1 in the environment loads the build with device-side range checks
# (libpreba_checked.so) instead: same entry points, slower kernels, for tests
_LIB_PATH = Path(__file__).resolve().parent / (
    "libpreba_checked.so" if os.environ.get("PREBA_CHECKED_BUILD") == "1" else "libpreba.so")

PACK_ALIGN = 128
SCRATCH_BYTES = 256
IMAGES_IN_PLACE = 1
IMAGES_OUT_IN_PLACE = 2
EX_ROUND_U8 = 1
OVERLAP_PREVIOUS = 1
F32, F16, BF16, U8 = 0, 1, 2, 3

OK = 0
ERR_INVALID_ARG = -1
ERR_BUFFER_TOO_SMALL = -2
ERR_BAD_TABLE = -3
ERR_CUDA = -4
ERR_TIMEOUT = -5
ERR_TOO_LARGE = -6
ERR_BAD_CROP = -7
ERR_RANGE = -8
ERR_UNSUPPORTED = -9
ERR_BAD_STREAM = -10
NOALLOC_MAX_BYTES = 64 << 20

EXPORTS = ("preba_query", "preba_pack", "preba_preprocess", "preba_preprocess_ex",
           "preba_preprocess_antialias", "preba_preprocess_host",
           "preba_preprocess_images",
           "preba_preprocess_host_noalloc", "preba_preprocess_repeated", "preba_serve_run",
           "preba_selftest_wait_limit",
           "preba_strerror",
           "preba_last_cuda_error",
           "preba_batching_params", "preba_batcher_create", "preba_batcher_destroy",
           "preba_batcher_push", "preba_batcher_poll",
           "preba_bucket_batcher_create", "preba_bucket_batcher_destroy",
           "preba_bucket_batcher_push", "preba_bucket_batcher_poll",
           "preba_audio_query", "preba_audio_pack", "preba_audio_logmel",
           "preba_audio_layout", "preba_audio_resample_query", "preba_audio_resample",
           "preba_jpeg_query", "preba_jpeg_decode")


class PrebaImg(ctypes.Structure):
    _fields_ = [("offset", ctypes.c_uint64), ("h", ctypes.c_uint32), ("w", ctypes.c_uint32)]


class PrebaSizes(ctypes.Structure):
    _fields_ = [("packed_bytes", ctypes.c_uint64), ("table_bytes", ctypes.c_uint64),
                ("out_bytes", ctypes.c_uint64), ("align", ctypes.c_uint32),
                ("reserved", ctypes.c_uint32)]


class PrebaBatch(ctypes.Structure):
    _fields_ = [("pixels", ctypes.c_void_p), ("pixels_bytes", ctypes.c_uint64),
                ("table", ctypes.c_void_p), ("table_host", ctypes.c_void_p),
                ("n", ctypes.c_uint32), ("flags", ctypes.c_uint32),
                ("out", ctypes.c_void_p), ("out_bytes", ctypes.c_uint64),
                ("status", ctypes.c_void_p), ("scratch", ctypes.c_void_p)]


class PrebaHostBatch(ctypes.Structure):
    _fields_ = [("packed_host", ctypes.c_void_p), ("packed_bytes", ctypes.c_uint64),
                ("table_host", ctypes.c_void_p), ("n", ctypes.c_uint32),
                ("reserved", ctypes.c_uint32), ("out_host", ctypes.c_void_p),
                ("out_bytes", ctypes.c_uint64), ("dev_pixels", ctypes.c_void_p),
                ("dev_table", ctypes.c_void_p), ("dev_out", ctypes.c_void_p),
                ("dev_status", ctypes.c_void_p), ("dev_scratch", ctypes.c_void_p)]


class PrebaOptions(ctypes.Structure):
    _fields_ = [("out_size", ctypes.c_uint32), ("resize_short", ctypes.c_uint32),
                ("mean", ctypes.c_float * 3), ("std", ctypes.c_float * 3),
                ("out_dtype", ctypes.c_int32), ("flags", ctypes.c_uint32),
                ("crop_origin", ctypes.c_void_p), ("crop_origin_host", ctypes.c_void_p)]


class PrebaImageBatch(ctypes.Structure):
    _fields_ = [("images", ctypes.c_void_p), ("h", ctypes.c_void_p), ("w", ctypes.c_void_p),
                ("n", ctypes.c_uint32), ("flags", ctypes.c_uint32),
                ("table_host", ctypes.c_void_p), ("out_host", ctypes.c_void_p),
                ("out_bytes", ctypes.c_uint64), ("dev_pixels", ctypes.c_void_p),
                ("dev_pixels_bytes", ctypes.c_uint64), ("dev_table", ctypes.c_void_p),
                ("dev_out", ctypes.c_void_p), ("dev_status", ctypes.c_void_p),
                ("dev_scratch", ctypes.c_void_p)]


class PrebaServe(ctypes.Structure):
    _fields_ = [("arrival_ns", ctypes.c_void_p), ("image_index", ctypes.c_void_p),
                ("n_requests", ctypes.c_uint32), ("pool_size", ctypes.c_uint32),
                ("pool_images", ctypes.c_void_p), ("pool_h", ctypes.c_void_p),
                ("pool_w", ctypes.c_void_p), ("batch_max", ctypes.c_uint32),
                ("n_servers", ctypes.c_uint32), ("time_queue_ns", ctypes.c_uint64),
                ("out_size", ctypes.c_uint32), ("resize_short", ctypes.c_uint32),
                ("mean", ctypes.c_float * 3), ("std", ctypes.c_float * 3),
                ("out_dtype", ctypes.c_int32), ("device", ctypes.c_int32),
                ("table_host", ctypes.c_void_p), ("out_host", ctypes.c_void_p),
                ("dev_table", ctypes.c_void_p), ("dev_out", ctypes.c_void_p),
                ("dev_status", ctypes.c_void_p), ("dev_scratch", ctypes.c_void_p),
                ("streams", ctypes.c_void_p), ("out_arena", ctypes.c_void_p),
                ("done_ns", ctypes.c_void_p), ("batch_size", ctypes.c_void_p),
                ("batch_first", ctypes.c_void_p), ("batch_release_ns", ctypes.c_void_p),
                ("batch_server", ctypes.c_void_p)]


class PrebaJpegSizes(ctypes.Structure):
    _fields_ = [("stage_bytes", ctypes.c_uint64), ("coef_bytes", ctypes.c_uint64),
                ("packed_bytes", ctypes.c_uint64), ("table_bytes", ctypes.c_uint64)]


class PrebaJpegBatch(ctypes.Structure):
    _fields_ = [("jpegs", ctypes.c_void_p), ("bytes", ctypes.c_void_p), ("n", ctypes.c_uint32),
                ("reserved", ctypes.c_uint32), ("stage_host", ctypes.c_void_p),
                ("stage_dev", ctypes.c_void_p), ("stage_bytes", ctypes.c_uint64),
                ("coef", ctypes.c_void_p), ("coef_bytes", ctypes.c_uint64),
                ("pixels", ctypes.c_void_p), ("pixels_bytes", ctypes.c_uint64),
                ("table", ctypes.c_void_p), ("table_host", ctypes.c_void_p),
                ("status", ctypes.c_void_p)]


class PrebaAudioSizes(ctypes.Structure):
    _fields_ = [("packed_samples", ctypes.c_uint64), ("table_bytes", ctypes.c_uint64),
                ("out_bytes", ctypes.c_uint64), ("t_max", ctypes.c_uint32),
                ("reserved", ctypes.c_uint32)]


class PrebaAudioBatch(ctypes.Structure):
    _fields_ = [("samples", ctypes.c_void_p), ("samples_count", ctypes.c_uint64),
                ("table", ctypes.c_void_p), ("table_host", ctypes.c_void_p),
                ("n", ctypes.c_uint32), ("t_max", ctypes.c_uint32),
                ("out", ctypes.c_void_p), ("out_bytes", ctypes.c_uint64),
                ("status", ctypes.c_void_p)]


UTT_DTYPE = np.dtype([("offset", "<u8"), ("length", "<u4"), ("frames", "<u4")])
AUDIO_MELS = 80
TABLE_DTYPE = np.dtype([("offset", "<u8"), ("h", "<u4"), ("w", "<u4")])


class PrebaError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        text = lib().preba_strerror(code).decode()
        extra = f" (cudaError {lib().preba_last_cuda_error()})" if code == ERR_CUDA else ""
        super().__init__(f"{where}: {text} [{code}]{extra}")


_lib = None


def lib() -> ctypes.CDLL:
    """The loaded library; raises if it is missing."""
    global _lib
    if _lib is None:
        if not _LIB_PATH.exists():
            raise RuntimeError(
                f"{_LIB_PATH} is missing: build it with "
                "`python -m paper_2411_19114_b200.build` (there is no CPU fallback)")
        L = ctypes.CDLL(str(_LIB_PATH))
        u32p = ctypes.POINTER(ctypes.c_uint32)
        f32p = ctypes.POINTER(ctypes.c_float)
        L.preba_query.argtypes = [u32p, u32p, ctypes.c_uint32, ctypes.c_uint32, ctypes.c_int,
                                  ctypes.POINTER(PrebaSizes)]
        L.preba_pack.argtypes = [ctypes.POINTER(ctypes.c_void_p), u32p, u32p, ctypes.c_uint32,
                                 ctypes.c_void_p, ctypes.c_uint64, ctypes.c_void_p]
        L.preba_preprocess.argtypes = [ctypes.POINTER(PrebaBatch), ctypes.c_uint32,
                                       ctypes.c_uint32, f32p, f32p, ctypes.c_int, ctypes.c_void_p]
        L.preba_preprocess_host.argtypes = [ctypes.POINTER(PrebaHostBatch), ctypes.c_uint32,
                                            ctypes.c_uint32, f32p, f32p, ctypes.c_int,
                                            ctypes.c_void_p]
        L.preba_preprocess_ex.argtypes = [ctypes.POINTER(PrebaBatch), ctypes.POINTER(PrebaOptions),
                                          ctypes.c_void_p]
        L.preba_preprocess_ex.restype = ctypes.c_int
        L.preba_preprocess_antialias.argtypes = L.preba_preprocess_ex.argtypes
        L.preba_preprocess_antialias.restype = ctypes.c_int
        L.preba_preprocess_images.argtypes = [ctypes.POINTER(PrebaImageBatch), ctypes.c_uint32,
                                              ctypes.c_uint32, f32p, f32p, ctypes.c_int,
                                              ctypes.c_void_p]
        L.preba_preprocess_images.restype = ctypes.c_int
        L.preba_preprocess_repeated.argtypes = [ctypes.POINTER(PrebaBatch), ctypes.c_uint32,
                                                ctypes.c_uint32, f32p, f32p, ctypes.c_int,
                                                ctypes.c_void_p, ctypes.c_uint32, f32p, f32p]
        L.preba_preprocess_repeated.restype = ctypes.c_int
        L.preba_serve_run.argtypes = [ctypes.POINTER(PrebaServe), ctypes.POINTER(ctypes.c_uint32)]
        L.preba_serve_run.restype = ctypes.c_int
        L.preba_selftest_wait_limit.argtypes = [ctypes.c_void_p, ctypes.c_void_p]
        L.preba_selftest_wait_limit.restype = ctypes.c_int
        L.preba_preprocess_host_noalloc.argtypes = [
            ctypes.c_void_p, ctypes.c_uint64, ctypes.c_void_p, ctypes.c_uint32, ctypes.c_void_p,
            ctypes.c_uint64, ctypes.c_void_p, ctypes.c_uint32, ctypes.c_uint32, f32p, f32p,
            ctypes.c_int, ctypes.c_void_p]
        L.preba_preprocess_host_noalloc.restype = ctypes.c_int
        u64p = ctypes.POINTER(ctypes.c_uint64)
        L.preba_batching_params.argtypes = [ctypes.c_uint32, ctypes.c_uint64, ctypes.c_uint32,
                                            u32p, u64p]
        L.preba_batching_params.restype = ctypes.c_int
        L.preba_batcher_create.argtypes = [ctypes.c_uint32, ctypes.c_uint64]
        L.preba_batcher_create.restype = ctypes.c_void_p
        L.preba_batcher_destroy.argtypes = [ctypes.c_void_p]
        L.preba_batcher_destroy.restype = None
        L.preba_batcher_push.argtypes = [ctypes.c_void_p, ctypes.c_uint64, ctypes.c_uint64]
        L.preba_batcher_push.restype = ctypes.c_int
        L.preba_batcher_poll.argtypes = [ctypes.c_void_p, ctypes.c_uint64, u64p, ctypes.c_uint32,
                                         u64p]
        L.preba_batcher_poll.restype = ctypes.c_int
        L.preba_audio_query.argtypes = [u32p, ctypes.c_uint32, ctypes.POINTER(PrebaAudioSizes)]
        L.preba_audio_query.restype = ctypes.c_int
        L.preba_audio_pack.argtypes = [ctypes.POINTER(ctypes.c_void_p), u32p, ctypes.c_uint32,
                                       ctypes.c_void_p, ctypes.c_uint64, ctypes.c_void_p]
        L.preba_audio_pack.restype = ctypes.c_int
        L.preba_audio_logmel.argtypes = [ctypes.POINTER(PrebaAudioBatch), ctypes.c_int,
                                         ctypes.c_void_p]
        L.preba_audio_logmel.restype = ctypes.c_int
        L.preba_bucket_batcher_create.argtypes = [ctypes.c_uint32, ctypes.c_uint64, u32p,
                                                  ctypes.c_uint64]
        L.preba_bucket_batcher_create.restype = ctypes.c_void_p
        L.preba_bucket_batcher_destroy.argtypes = [ctypes.c_void_p]
        L.preba_bucket_batcher_destroy.restype = None
        L.preba_bucket_batcher_push.argtypes = [ctypes.c_void_p, ctypes.c_uint64, ctypes.c_uint64,
                                                ctypes.c_uint64]
        L.preba_bucket_batcher_push.restype = ctypes.c_int
        L.preba_bucket_batcher_poll.argtypes = [ctypes.c_void_p, ctypes.c_uint64, u64p,
                                                ctypes.c_uint32, u64p]
        L.preba_bucket_batcher_poll.restype = ctypes.c_int
        L.preba_audio_layout.argtypes = [u32p, ctypes.c_uint32, ctypes.c_void_p]
        L.preba_audio_layout.restype = ctypes.c_int
        L.preba_audio_resample_query.argtypes = [u32p, ctypes.c_uint32, ctypes.c_uint32,
                                                 ctypes.c_uint32, u32p]
        L.preba_audio_resample_query.restype = ctypes.c_int
        L.preba_audio_resample.argtypes = [ctypes.c_void_p, ctypes.c_uint64, ctypes.c_void_p,
                                           ctypes.c_void_p, ctypes.c_uint64, ctypes.c_void_p,
                                           ctypes.c_uint32, ctypes.c_uint32, ctypes.c_uint32,
                                           ctypes.c_uint32, ctypes.c_void_p, ctypes.c_void_p]
        L.preba_audio_resample.restype = ctypes.c_int
        L.preba_jpeg_query.argtypes = [ctypes.POINTER(ctypes.c_void_p), u64p, ctypes.c_uint32, u32p,
                                       u32p, ctypes.POINTER(PrebaJpegSizes)]
        L.preba_jpeg_query.restype = ctypes.c_int
        L.preba_jpeg_decode.argtypes = [ctypes.POINTER(PrebaJpegBatch), ctypes.c_void_p]
        L.preba_jpeg_decode.restype = ctypes.c_int
        L.preba_strerror.argtypes = [ctypes.c_int]
        L.preba_strerror.restype = ctypes.c_char_p
        L.preba_last_cuda_error.argtypes = []
        for name in ("preba_query", "preba_pack", "preba_preprocess", "preba_preprocess_host",
                     "preba_last_cuda_error"):
            getattr(L, name).restype = ctypes.c_int
        _lib = L
    return _lib


def _u32(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.uint32))


def _f3(v):
    a = np.ascontiguousarray(np.asarray(v, dtype=np.float32))
    if a.shape != (3,):
        raise ValueError("mean/std must have 3 entries")
    return a


def _p(a: np.ndarray, ctype):
    return a.ctypes.data_as(ctypes.POINTER(ctype))


def preba_strerror(code: int) -> str:
    return lib().preba_strerror(code).decode()


def preba_query(h, w, out_size: int, out_dtype: int) -> PrebaSizes:
    h, w = _u32(h), _u32(w)
    sizes = PrebaSizes()
    rc = lib().preba_query(_p(h, ctypes.c_uint32), _p(w, ctypes.c_uint32), len(h), out_size,
                           out_dtype, ctypes.byref(sizes))
    if rc != OK:
        raise PrebaError(rc, "preba_query")
    return sizes


def preba_pack(images, packed: np.ndarray | None = None, table: np.ndarray | None = None):
    """Pack a list of HWC uint8 arrays.  ``packed``/``table`` may be caller-provided
    (e.g. views of pinned memory); returns (packed, table)."""
    imgs = [np.ascontiguousarray(im, dtype=np.uint8) for im in images]
    n = len(imgs)
    for im in imgs:
        if im.ndim != 3 or im.shape[2] != 3:
            raise ValueError("images must be HWC with 3 channels")
    h = _u32([im.shape[0] for im in imgs])
    w = _u32([im.shape[1] for im in imgs])
    if packed is None:
        total = preba_query(h, w, 1, F32).packed_bytes
        packed = np.empty(total, dtype=np.uint8)
    if table is None:
        table = np.zeros(n, dtype=TABLE_DTYPE)
    if packed.dtype != np.uint8 or not packed.flags.c_contiguous:
        raise ValueError("packed must be a contiguous uint8 array")
    if table.dtype != TABLE_DTYPE or len(table) < n or not table.flags.c_contiguous:
        raise ValueError("table must be a contiguous TABLE_DTYPE array with n entries")
    ptrs = (ctypes.c_void_p * n)(*[im.ctypes.data for im in imgs])
    rc = lib().preba_pack(ptrs, _p(h, ctypes.c_uint32), _p(w, ctypes.c_uint32), n,
                          packed.ctypes.data, packed.nbytes, table.ctypes.data)
    if rc != OK:
        raise PrebaError(rc, "preba_pack")
    return packed, table


def preba_preprocess(pixels, table, n: int, out, out_size: int, resize_short: int, mean, std,
                     out_dtype: int, stream=None, table_host: np.ndarray | None = None,
                     status=None, pixels_bytes: int | None = None,
                     out_bytes: int | None = None, scratch=None, flags: int = 0) -> None:
    """``pixels``, ``table``, ``out`` and ``status`` are CUDA tensors (or raw device
    addresses); ``stream`` is a torch stream, a raw cudaStream_t or None for torch's
    current stream."""
    import torch

    def addr(t):
        return int(t) if isinstance(t, int) else t.data_ptr()

    def nbytes(t, given):
        if given is not None:
            return given
        return t.numel() * t.element_size()

    if stream is None:
        stream = torch.cuda.current_stream().cuda_stream
    elif hasattr(stream, "cuda_stream"):
        stream = stream.cuda_stream
    batch = PrebaBatch()
    batch.pixels = addr(pixels)
    batch.pixels_bytes = nbytes(pixels, pixels_bytes)
    batch.table = addr(table)
    batch.table_host = table_host.ctypes.data if table_host is not None else None
    batch.n = n
    batch.out = addr(out)
    batch.out_bytes = nbytes(out, out_bytes)
    batch.status = addr(status) if status is not None else None
    batch.scratch = addr(scratch) if scratch is not None else None
    batch.flags = flags
    m, s = _f3(mean), _f3(std)
    rc = lib().preba_preprocess(ctypes.byref(batch), out_size, resize_short,
                                _p(m, ctypes.c_float), _p(s, ctypes.c_float), out_dtype,
                                ctypes.c_void_p(stream))
    if rc != OK:
        raise PrebaError(rc, "preba_preprocess")


class PreparedPreprocessEx:
    """The arguments of one ``preba_preprocess_ex`` call, marshalled once (see
    ``preba_preprocess_ex``); calling the object makes the foreign call and nothing else."""

    def __init__(self, pixels, table, n: int, out, out_size: int, resize_short: int, mean, std,
                 out_dtype: int, round_u8: bool = False, crop_origin=None,
                 crop_origin_host: np.ndarray | None = None, stream=None,
                 table_host: np.ndarray | None = None, status=None, scratch=None,
                 flags: int = 0, entry: str = "preba_preprocess_ex"):
        import torch

        if stream is None:
            stream = torch.cuda.current_stream().cuda_stream
        elif hasattr(stream, "cuda_stream"):
            stream = stream.cuda_stream
        self._entry = entry
        self._fn = getattr(lib(), entry)
        batch = PrebaBatch()
        batch.pixels = pixels.data_ptr()
        batch.pixels_bytes = pixels.numel() * pixels.element_size()
        batch.table = table.data_ptr()
        batch.table_host = table_host.ctypes.data if table_host is not None else None
        batch.n = n
        batch.out = out.data_ptr()
        batch.out_bytes = out.numel() * out.element_size()
        batch.status = status.data_ptr() if status is not None else None
        batch.scratch = scratch.data_ptr() if scratch is not None else None
        batch.flags = flags
        opt = PrebaOptions()
        opt.out_size, opt.resize_short = out_size, resize_short
        opt.mean = (ctypes.c_float * 3)(*[float(v) for v in _f3(mean)])
        opt.std = (ctypes.c_float * 3)(*[float(v) for v in _f3(std)])
        opt.out_dtype = out_dtype
        opt.flags = EX_ROUND_U8 if round_u8 else 0
        opt.crop_origin = crop_origin.data_ptr() if crop_origin is not None else None
        if crop_origin_host is not None:
            crop_origin_host = np.ascontiguousarray(crop_origin_host, dtype=np.uint32)
            opt.crop_origin_host = crop_origin_host.ctypes.data
        self._keep = (pixels, table, out, status, scratch, table_host, crop_origin,
                      crop_origin_host, batch, opt)
        self._args = (ctypes.byref(batch), ctypes.byref(opt), ctypes.c_void_p(stream))

    def __call__(self) -> None:
        rc = self._fn(*self._args)
        if rc != OK:
            raise PrebaError(rc, self._entry)


def preba_preprocess_ex(pixels, table, n: int, out, out_size: int, resize_short: int, mean, std,
                        out_dtype: int, round_u8: bool = False, crop_origin=None,
                        crop_origin_host: np.ndarray | None = None, stream=None,
                        table_host: np.ndarray | None = None, status=None, scratch=None,
                        flags: int = 0) -> None:
    """``preba_preprocess`` with a crop window per image (``crop_origin``: CUDA int32/uint32
    tensor of 2n values (top, left); ``crop_origin_host``: uint32 array for the host check) and
    optional rounding of the resized pixel to uint8 (``out_dtype`` U8 writes it as [n,C,C,3])."""
    PreparedPreprocessEx(pixels, table, n, out, out_size, resize_short, mean, std, out_dtype,
                         round_u8, crop_origin, crop_origin_host, stream, table_host, status,
                         scratch, flags)()


def preba_preprocess_antialias(pixels, table, n: int, out, out_size: int, resize_short: int, mean,
                               std, out_dtype: int, crop_origin=None,
                               crop_origin_host: np.ndarray | None = None, stream=None,
                               table_host: np.ndarray | None = None, status=None) -> None:
    """``preba_preprocess_antialias``: the transform with the triangle filter widened by the
    reduction factor; arguments as ``preba_preprocess_ex`` without rounding."""
    PreparedPreprocessEx(pixels, table, n, out, out_size, resize_short, mean, std, out_dtype,
                         False, crop_origin, crop_origin_host, stream, table_host, status,
                         None, 0, entry="preba_preprocess_antialias")()


class PreparedPreprocess:
    """The arguments of one ``preba_preprocess`` call, marshalled once; calling the object
    makes the foreign call and nothing else (for loops that launch back to back)."""

    def __init__(self, pixels, table, n: int, out, out_size: int, resize_short: int, mean, std,
                 out_dtype: int, stream=None, table_host: np.ndarray | None = None, status=None,
                 scratch=None, flags: int = 0):
        import torch

        if stream is None:
            stream = torch.cuda.current_stream().cuda_stream
        elif hasattr(stream, "cuda_stream"):
            stream = stream.cuda_stream
        self._keep = (pixels, table, out, status, table_host, scratch)
        b = PrebaBatch()
        b.pixels = pixels.data_ptr()
        b.pixels_bytes = pixels.numel() * pixels.element_size()
        b.table = table.data_ptr()
        b.table_host = table_host.ctypes.data if table_host is not None else None
        b.n = n
        b.out = out.data_ptr()
        b.out_bytes = out.numel() * out.element_size()
        b.status = status.data_ptr() if status is not None else None
        b.scratch = scratch.data_ptr() if scratch is not None else None
        b.flags = flags
        self._batch = b
        self._mean, self._std = _f3(mean), _f3(std)
        self._args = (ctypes.byref(b), out_size, resize_short, _p(self._mean, ctypes.c_float),
                      _p(self._std, ctypes.c_float), out_dtype, ctypes.c_void_p(stream))
        self._fn = lib().preba_preprocess

    def __call__(self) -> None:
        rc = self._fn(*self._args)
        if rc != OK:
            raise PrebaError(rc, "preba_preprocess")

    def repeated(self, iterations: int) -> tuple[np.ndarray, float]:
        """``preba_preprocess_repeated``: (device time of every launch in us, span in ms).
        Blocks until the stream is done; the interpreter lock is released meanwhile."""
        lat = np.zeros(iterations, dtype=np.float32)
        span = ctypes.c_float()
        rc = lib().preba_preprocess_repeated(*self._args, iterations, _p(lat, ctypes.c_float),
                                             ctypes.byref(span))
        if rc != OK:
            raise PrebaError(rc, "preba_preprocess_repeated")
        return lat, span.value


def preba_preprocess_host(packed_host, table_host: np.ndarray, n: int, out_host, dev_pixels,
                          dev_table, dev_out, out_size: int, resize_short: int, mean, std,
                          out_dtype: int, stream=None, dev_status=None, dev_scratch=None) -> None:
    """``packed_host``/``out_host`` are (pinned) CPU tensors or numpy arrays; ``dev_*`` are
    CUDA tensors used as staging."""
    import torch

    def haddr(t):
        return t.ctypes.data if isinstance(t, np.ndarray) else t.data_ptr()

    def hbytes(t):
        return t.nbytes if isinstance(t, np.ndarray) else t.numel() * t.element_size()

    if stream is None:
        stream = torch.cuda.current_stream().cuda_stream
    elif hasattr(stream, "cuda_stream"):
        stream = stream.cuda_stream
    b = PrebaHostBatch()
    b.packed_host = haddr(packed_host)
    b.packed_bytes = hbytes(packed_host)
    b.table_host = table_host.ctypes.data
    b.n = n
    b.out_host = haddr(out_host)
    b.out_bytes = hbytes(out_host)
    if dev_pixels.numel() * dev_pixels.element_size() < b.packed_bytes:
        raise PrebaError(ERR_BUFFER_TOO_SMALL, "preba_preprocess_host (dev_pixels)")
    if dev_out.numel() * dev_out.element_size() < b.out_bytes:
        raise PrebaError(ERR_BUFFER_TOO_SMALL, "preba_preprocess_host (dev_out)")
    b.dev_pixels = dev_pixels.data_ptr()
    b.dev_table = dev_table.data_ptr()
    b.dev_out = dev_out.data_ptr()
    b.dev_status = dev_status.data_ptr() if dev_status is not None else None
    b.dev_scratch = dev_scratch.data_ptr() if dev_scratch is not None else None
    m, s = _f3(mean), _f3(std)
    rc = lib().preba_preprocess_host(ctypes.byref(b), out_size, resize_short,
                                     _p(m, ctypes.c_float), _p(s, ctypes.c_float), out_dtype,
                                     ctypes.c_void_p(stream))
    if rc != OK:
        raise PrebaError(rc, "preba_preprocess_host")


class PreparedImages:
    """The arguments of ``preba_preprocess_images`` for a fixed set of host images, marshalled
    once.  ``images`` are uint8 HWC arrays or CPU tensors (pinned for asynchronous copies);
    ``table_host`` is a pinned CPU tensor of ``16 * n`` bytes that every call rewrites;
    ``out_host`` a (pinned) CPU tensor; ``dev_*`` CUDA tensors used as staging.  With
    ``in_place`` the kernel reads the (pinned, 128-byte aligned) images over the link itself
    and ``dev_pixels`` may be None; with ``out_in_place`` it writes the (pinned) ``out_host``
    itself and ``dev_out`` may be None."""

    def __init__(self, images, table_host, out_host, dev_pixels, dev_table, dev_out,
                 out_size: int, resize_short: int, mean, std, out_dtype: int, stream=None,
                 dev_status=None, dev_scratch=None, in_place: bool = False,
                 out_in_place: bool = False):
        import torch

        def haddr(t):
            return t.ctypes.data if isinstance(t, np.ndarray) else t.data_ptr()

        def hbytes(t):
            return t.nbytes if isinstance(t, np.ndarray) else t.numel() * t.element_size()

        if stream is None:
            stream = torch.cuda.current_stream().cuda_stream
        elif hasattr(stream, "cuda_stream"):
            stream = stream.cuda_stream
        n = len(images)
        for im in images:
            if tuple(im.shape)[2:] != (3,) or hbytes(im) != im.shape[0] * im.shape[1] * 3:
                raise ValueError("images must be contiguous uint8 arrays of shape (h, w, 3)")
        self._ptrs = (ctypes.c_void_p * n)(*[haddr(im) for im in images])
        self._h = _u32([im.shape[0] for im in images])
        self._w = _u32([im.shape[1] for im in images])
        if hbytes(table_host) < 16 * n:
            raise PrebaError(ERR_BUFFER_TOO_SMALL, "preba_preprocess_images (table_host)")
        b = PrebaImageBatch()
        b.images = ctypes.cast(self._ptrs, ctypes.c_void_p)
        b.h, b.w, b.n = self._h.ctypes.data, self._w.ctypes.data, n
        b.table_host = haddr(table_host)
        b.out_host, b.out_bytes = haddr(out_host), hbytes(out_host)
        b.flags = (IMAGES_IN_PLACE if in_place else 0) | (IMAGES_OUT_IN_PLACE if out_in_place else 0)
        if dev_pixels is not None:
            b.dev_pixels = dev_pixels.data_ptr()
            b.dev_pixels_bytes = dev_pixels.numel() * dev_pixels.element_size()
        b.dev_table = dev_table.data_ptr()
        if dev_out is not None:
            b.dev_out = dev_out.data_ptr()
            if dev_out.numel() * dev_out.element_size() < b.out_bytes:
                raise PrebaError(ERR_BUFFER_TOO_SMALL, "preba_preprocess_images (dev_out)")
        elif not out_in_place:
            raise ValueError("dev_out is needed unless the kernel writes the result in place")
        b.dev_status = dev_status.data_ptr() if dev_status is not None else None
        b.dev_scratch = dev_scratch.data_ptr() if dev_scratch is not None else None
        self._b, self._m, self._s = b, _f3(mean), _f3(std)
        self._keep = (images, table_host, out_host, dev_pixels, dev_table, dev_out, dev_status,
                      dev_scratch)
        self._args = (ctypes.byref(b), out_size, resize_short, _p(self._m, ctypes.c_float),
                      _p(self._s, ctypes.c_float), out_dtype, ctypes.c_void_p(stream))

    def __call__(self) -> None:
        rc = lib().preba_preprocess_images(*self._args)
        if rc != OK:
            raise PrebaError(rc, "preba_preprocess_images")


def preba_preprocess_host_noalloc(packed_host, table_host: np.ndarray, n: int, out_host,
                                  out_size: int, resize_short: int, mean, std, out_dtype: int,
                                  stream=None, status_host=None) -> None:
    """Host buffers in, host buffers out, staged through the array the library carries in
    device memory: nothing is allocated.  ``packed_host``/``out_host``/``status_host`` are
    (pinned) CPU tensors or numpy arrays.  Calls must not overlap on the device."""
    import torch

    def haddr(t):
        return t.ctypes.data if isinstance(t, np.ndarray) else t.data_ptr()

    def hbytes(t):
        return t.nbytes if isinstance(t, np.ndarray) else t.numel() * t.element_size()

    if stream is None:
        stream = torch.cuda.current_stream().cuda_stream
    elif hasattr(stream, "cuda_stream"):
        stream = stream.cuda_stream
    m, s = _f3(mean), _f3(std)
    rc = lib().preba_preprocess_host_noalloc(
        haddr(packed_host), hbytes(packed_host), table_host.ctypes.data, n, haddr(out_host),
        hbytes(out_host), haddr(status_host) if status_host is not None else None, out_size,
        resize_short, _p(m, ctypes.c_float), _p(s, ctypes.c_float), out_dtype,
        ctypes.c_void_p(stream))
    if rc != OK:
        raise PrebaError(rc, "preba_preprocess_host_noalloc")


def preba_serve_run(arrival_ns, image_index, pool_images, batch_max: int, time_queue_ns: int,
                    servers, out_size: int, resize_short: int, mean, std, out_dtype: int,
                    out_arena=None, device: int = 0) -> dict:
    """``preba_serve_run``: requests ``i`` arriving at ``arrival_ns[i]`` (ns from the start of the
    run) carry pool image ``image_index[i]``; ``pool_images`` are pinned, 128-byte aligned uint8
    CPU tensors (h, w, 3); ``servers`` is a list of dicts with the staging of one server each:
    ``table_host`` (pinned uint8, 16 bytes per image of a full batch), ``out_host`` (pinned),
    ``dev_table``, ``dev_out``, optional ``dev_status`` and ``dev_scratch`` (CUDA tensors) and
    ``stream``.  Blocks until every request is served (the interpreter lock is released).
    Returns the completion time of every request and the record of the batches."""
    arr = np.ascontiguousarray(np.asarray(arrival_ns, dtype=np.uint64))
    idx = _u32(image_index)
    n, k, v = len(arr), len(pool_images), len(servers)
    ptrs = (ctypes.c_void_p * k)(*[im.data_ptr() for im in pool_images])
    ph = _u32([im.shape[0] for im in pool_images])
    pw = _u32([im.shape[1] for im in pool_images])

    def column(name, optional=False):
        vals = []
        for sv in servers:
            t = sv.get(name)
            if t is None and not optional:
                raise ValueError(f"server staging lacks {name}")
            if t is None:
                vals.append(None)
            elif name == "stream":
                vals.append(t.cuda_stream if hasattr(t, "cuda_stream") else int(t))
            else:
                vals.append(t.data_ptr())
        return (ctypes.c_void_p * v)(*vals)

    cols = {name: column(name, name in ("dev_status", "dev_scratch", "out_host"))
            for name in ("table_host", "out_host", "dev_table", "dev_out", "dev_status",
                         "dev_scratch", "stream")}
    done = np.zeros(n, dtype=np.uint64)
    b_size, b_first = np.zeros(n, dtype=np.uint32), np.zeros(n, dtype=np.uint32)
    b_release, b_server = np.zeros(n, dtype=np.uint64), np.zeros(n, dtype=np.uint32)
    sv = PrebaServe()
    sv.arrival_ns, sv.image_index = arr.ctypes.data, idx.ctypes.data
    sv.n_requests, sv.pool_size = n, k
    sv.pool_images = ctypes.cast(ptrs, ctypes.c_void_p)
    sv.pool_h, sv.pool_w = ph.ctypes.data, pw.ctypes.data
    sv.batch_max, sv.n_servers, sv.time_queue_ns = batch_max, v, time_queue_ns
    sv.out_size, sv.resize_short = out_size, resize_short
    sv.mean = (ctypes.c_float * 3)(*[float(x) for x in _f3(mean)])
    sv.std = (ctypes.c_float * 3)(*[float(x) for x in _f3(std)])
    sv.out_dtype, sv.device = out_dtype, device
    sv.table_host = ctypes.cast(cols["table_host"], ctypes.c_void_p)
    sv.out_host = ctypes.cast(cols["out_host"], ctypes.c_void_p)
    sv.dev_table = ctypes.cast(cols["dev_table"], ctypes.c_void_p)
    sv.dev_out = ctypes.cast(cols["dev_out"], ctypes.c_void_p)
    sv.dev_status = ctypes.cast(cols["dev_status"], ctypes.c_void_p)
    sv.dev_scratch = ctypes.cast(cols["dev_scratch"], ctypes.c_void_p)
    sv.streams = ctypes.cast(cols["stream"], ctypes.c_void_p)
    sv.out_arena = out_arena.data_ptr() if out_arena is not None else None
    sv.done_ns = done.ctypes.data
    sv.batch_size, sv.batch_first = b_size.ctypes.data, b_first.ctypes.data
    sv.batch_release_ns, sv.batch_server = b_release.ctypes.data, b_server.ctypes.data
    nb = ctypes.c_uint32()
    rc = lib().preba_serve_run(ctypes.byref(sv), ctypes.byref(nb))
    if rc != OK:
        raise PrebaError(rc, "preba_serve_run")
    m = nb.value
    order = np.argsort(b_first[:m], kind="stable")
    return {"done_ns": done, "batch_size": b_size[:m][order], "batch_first": b_first[:m][order],
            "batch_release_ns": b_release[:m][order], "batch_server": b_server[:m][order]}


def preba_selftest_wait_limit(status, stream=None) -> None:
    """``status`` is a zeroed CUDA int32 tensor; after the stream has run it holds ERR_TIMEOUT."""
    import torch

    if stream is None:
        stream = torch.cuda.current_stream().cuda_stream
    elif hasattr(stream, "cuda_stream"):
        stream = stream.cuda_stream
    rc = lib().preba_selftest_wait_limit(status.data_ptr(), ctypes.c_void_p(stream))
    if rc != OK:
        raise PrebaError(rc, "preba_selftest_wait_limit")


NEVER = (1 << 64) - 1


def preba_batching_params(batch_knee: int, time_knee_ns: int, n_servers: int) -> tuple[int, int]:
    bm, tq = ctypes.c_uint32(), ctypes.c_uint64()
    rc = lib().preba_batching_params(batch_knee, time_knee_ns, n_servers, ctypes.byref(bm),
                                     ctypes.byref(tq))
    if rc != OK:
        raise PrebaError(rc, "preba_batching_params")
    return bm.value, tq.value


class PrebaBatcher:
    """A queue of the batching front-end (``preba_batcher_*``)."""

    def __init__(self, batch_max: int, time_queue_ns: int):
        self._h = lib().preba_batcher_create(batch_max, time_queue_ns)
        if not self._h:
            raise PrebaError(ERR_INVALID_ARG, "preba_batcher_create")
        self._ids = (ctypes.c_uint64 * batch_max)()
        self._cap = batch_max

    def push(self, request_id: int, arrival_ns: int) -> None:
        rc = lib().preba_batcher_push(self._h, request_id, arrival_ns)
        if rc != OK:
            raise PrebaError(rc, "preba_batcher_push")

    def poll(self, now_ns: int) -> tuple[list[int], int]:
        """(ids of the batch that is due, or []; next deadline or NEVER)."""
        nxt = ctypes.c_uint64()
        rc = lib().preba_batcher_poll(self._h, now_ns, self._ids, self._cap, ctypes.byref(nxt))
        if rc < 0:
            raise PrebaError(rc, "preba_batcher_poll")
        return [int(self._ids[i]) for i in range(rc)], nxt.value

    def close(self) -> None:
        if self._h:
            lib().preba_batcher_destroy(self._h)
            self._h = None

    def __del__(self):
        self.close()


# ---- audio path ------------------------------------------------------------------------------------

def preba_audio_query(lengths) -> PrebaAudioSizes:
    ln = _u32(lengths)
    sizes = PrebaAudioSizes()
    rc = lib().preba_audio_query(_p(ln, ctypes.c_uint32), len(ln), ctypes.byref(sizes))
    if rc != OK:
        raise PrebaError(rc, "preba_audio_query")
    return sizes


def preba_audio_pack(utterances, packed: np.ndarray | None = None,
                     table: np.ndarray | None = None):
    """Packed float32 sample buffer and {offset, length, frames} table of a list of 1-D
    float32 utterances."""
    utts = [np.ascontiguousarray(u, dtype=np.float32).reshape(-1) for u in utterances]
    n = len(utts)
    ln = _u32([u.size for u in utts])
    sizes = preba_audio_query(ln)
    if packed is None:
        packed = np.full(sizes.packed_samples, np.nan, dtype=np.float32)  # pack writes every sample
    if table is None:
        table = np.zeros(n, dtype=UTT_DTYPE)
    ptrs = (ctypes.c_void_p * n)(*[u.ctypes.data for u in utts])
    rc = lib().preba_audio_pack(ptrs, _p(ln, ctypes.c_uint32), n, packed.ctypes.data,
                                packed.size, table.ctypes.data)
    if rc != OK:
        raise PrebaError(rc, "preba_audio_pack")
    return packed, table


AUDIO_NORMALIZE, AUDIO_OVERLAP_PREVIOUS = 1, 2


class PreparedAudio:
    """The arguments of one ``preba_audio_logmel`` call, marshalled once.  ``samples``, ``table``,
    ``out`` (float32 [n, 80, t_max]) and ``status`` are CUDA tensors."""

    def __init__(self, samples, table, n: int, t_max: int, out, normalize: bool = True,
                 stream=None, table_host: np.ndarray | None = None, status=None,
                 overlap_previous: bool = False):
        import torch

        if stream is None:
            stream = torch.cuda.current_stream().cuda_stream
        elif hasattr(stream, "cuda_stream"):
            stream = stream.cuda_stream
        b = PrebaAudioBatch()
        b.samples, b.samples_count = samples.data_ptr(), samples.numel()
        b.table = table.data_ptr()
        b.table_host = table_host.ctypes.data if table_host is not None else None
        b.n, b.t_max = n, t_max
        b.out, b.out_bytes = out.data_ptr(), out.numel() * out.element_size()
        b.status = status.data_ptr() if status is not None else None
        self._keep = (samples, table, out, status, table_host, b)
        bits = (AUDIO_NORMALIZE if normalize else 0) | (AUDIO_OVERLAP_PREVIOUS if overlap_previous else 0)
        self._args = (ctypes.byref(b), bits, ctypes.c_void_p(stream))

    def __call__(self) -> None:
        rc = lib().preba_audio_logmel(*self._args)
        if rc != OK:
            raise PrebaError(rc, "preba_audio_logmel")


def preba_audio_logmel(samples, table, n: int, t_max: int, out, normalize: bool = True,
                       stream=None, table_host: np.ndarray | None = None, status=None) -> None:
    PreparedAudio(samples, table, n, t_max, out, normalize, stream, table_host, status)()


class BucketBatcher:
    """The batching front-end for variable-length inputs (``preba_bucket_batcher_*``)."""

    def __init__(self, window: int, batch_max, time_queue_ns: int):
        bm = _u32(batch_max)
        self._h = lib().preba_bucket_batcher_create(len(bm), window, _p(bm, ctypes.c_uint32),
                                                    time_queue_ns)
        if not self._h:
            raise PrebaError(ERR_INVALID_ARG, "preba_bucket_batcher_create")
        self._cap = int(bm.max())
        self._ids = (ctypes.c_uint64 * self._cap)()

    def push(self, request_id: int, arrival_ns: int, length: int) -> None:
        rc = lib().preba_bucket_batcher_push(self._h, request_id, arrival_ns, length)
        if rc != OK:
            raise PrebaError(rc, "preba_bucket_batcher_push")

    def poll(self, now_ns: int) -> tuple[list[int], int]:
        """(ids of one due batch or [], time at which the oldest waiting request runs out)."""
        nxt = ctypes.c_uint64()
        rc = lib().preba_bucket_batcher_poll(self._h, now_ns, self._ids, self._cap,
                                             ctypes.byref(nxt))
        if rc < 0:
            raise PrebaError(rc, "preba_bucket_batcher_poll")
        return [int(self._ids[i]) for i in range(rc)], int(nxt.value)

    def __del__(self):
        if getattr(self, "_h", None):
            lib().preba_bucket_batcher_destroy(self._h)
            self._h = None


def preba_audio_layout(lengths) -> np.ndarray:
    """The {offset, length, frames} table of a packed sample buffer for the given lengths."""
    ln = _u32(lengths)
    table = np.zeros(len(ln), dtype=UTT_DTYPE)
    rc = lib().preba_audio_layout(_p(ln, ctypes.c_uint32), len(ln), table.ctypes.data)
    if rc != OK:
        raise PrebaError(rc, "preba_audio_layout")
    return table


def preba_audio_resample_query(lengths_in, rate_in: int, rate_out: int) -> np.ndarray:
    ln = _u32(lengths_in)
    out = np.zeros(len(ln), dtype=np.uint32)
    rc = lib().preba_audio_resample_query(_p(ln, ctypes.c_uint32), len(ln), rate_in, rate_out,
                                          _p(out, ctypes.c_uint32))
    if rc != OK:
        raise PrebaError(rc, "preba_audio_resample_query")
    return out


def preba_audio_resample(samples_in, table_in, samples_out, table_out, n: int, longest_out: int,
                         rate_in: int, rate_out: int, status=None, stream=None) -> None:
    """``samples_*`` and ``table_*`` are CUDA tensors (packed float32 samples, tables as bytes)."""
    import torch

    if stream is None:
        stream = torch.cuda.current_stream().cuda_stream
    elif hasattr(stream, "cuda_stream"):
        stream = stream.cuda_stream
    rc = lib().preba_audio_resample(samples_in.data_ptr(), samples_in.numel(), table_in.data_ptr(),
                                    samples_out.data_ptr(), samples_out.numel(),
                                    table_out.data_ptr(), n, longest_out, rate_in, rate_out,
                                    status.data_ptr() if status is not None else None,
                                    ctypes.c_void_p(stream))
    if rc != OK:
        raise PrebaError(rc, "preba_audio_resample")


# ---- JPEG Decode ---------------------------------------------------------------------------------------

def _streams(jpegs):
    """The streams as contiguous uint8 arrays, their pointer array and their sizes."""
    arrs = [np.frombuffer(j, dtype=np.uint8) if isinstance(j, (bytes, bytearray, memoryview))
            else np.ascontiguousarray(j, dtype=np.uint8) for j in jpegs]
    ptrs = (ctypes.c_void_p * len(arrs))(*[a.ctypes.data for a in arrs])
    sizes = np.ascontiguousarray([a.size for a in arrs], dtype=np.uint64)
    return arrs, ptrs, sizes


def preba_jpeg_query(jpegs):
    """(heights, widths, PrebaJpegSizes) of a list of JPEG streams (bytes or uint8 arrays)."""
    arrs, ptrs, sizes = _streams(jpegs)
    n = len(arrs)
    h, w = np.zeros(n, dtype=np.uint32), np.zeros(n, dtype=np.uint32)
    out = PrebaJpegSizes()
    rc = lib().preba_jpeg_query(ptrs, _p(sizes, ctypes.c_uint64), n, _p(h, ctypes.c_uint32),
                                _p(w, ctypes.c_uint32), ctypes.byref(out))
    if rc != OK:
        raise PrebaError(rc, "preba_jpeg_query")
    return h, w, out


class PreparedJpeg:
    """The arguments of ``preba_jpeg_decode`` for a fixed list of streams, marshalled once.
    ``stage_host`` and ``table_host`` are pinned CPU uint8 tensors, ``stage_dev``, ``coef`` (int16),
    ``pixels`` (uint8), ``table`` (uint8, 16 bytes per image) and ``status`` CUDA tensors, sized
    by ``preba_jpeg_query``."""

    def __init__(self, jpegs, stage_host, stage_dev, coef, pixels, table, table_host, status=None,
                 stream=None):
        import torch

        if stream is None:
            stream = torch.cuda.current_stream().cuda_stream
        elif hasattr(stream, "cuda_stream"):
            stream = stream.cuda_stream
        self._arrs, self._ptrs, self._sizes = _streams(jpegs)
        b = PrebaJpegBatch()
        b.jpegs = ctypes.cast(self._ptrs, ctypes.c_void_p)
        b.bytes = self._sizes.ctypes.data
        b.n = len(self._arrs)
        b.stage_host, b.stage_dev = stage_host.data_ptr(), stage_dev.data_ptr()
        b.stage_bytes = min(stage_host.numel(), stage_dev.numel())
        b.coef, b.coef_bytes = coef.data_ptr(), coef.numel() * coef.element_size()
        b.pixels, b.pixels_bytes = pixels.data_ptr(), pixels.numel() * pixels.element_size()
        b.table, b.table_host = table.data_ptr(), table_host.data_ptr()
        b.status = status.data_ptr() if status is not None else None
        self._keep = (stage_host, stage_dev, coef, pixels, table, table_host, status, b)
        self._args = (ctypes.byref(b), ctypes.c_void_p(stream))

    def __call__(self) -> None:
        rc = lib().preba_jpeg_decode(*self._args)
        if rc != OK:
            raise PrebaError(rc, "preba_jpeg_decode")
