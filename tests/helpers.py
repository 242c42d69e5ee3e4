"""Shared by the GPU tests: run a batch through the C ABI on the device, compare with the oracle."""
from __future__ import annotations

import os

import numpy as np

import oracle
from paper_2411_19114_b200 import binding as pb

MEAN = (0.485, 0.456, 0.406)
STD = (0.229, 0.224, 0.225)
GUARD = 4096
CANARY = 0xA5
FP32_TOL = 1e-5  # max abs error against the double oracle, fp32 output
FP16_ABS = 1e-5  # second clause of the fp16 criterion (see fp16_report)


def host_threads() -> int:
    return max(1, len(os.sched_getaffinity(0)))


def run_gpu(images, c, s, mean=MEAN, std=STD, out_dtype=pb.F32, stream=None,
            check_host_table=True, dynamic=True):
    """Pack on the host, copy to the device between guard bands, run, return the result
    as a numpy array [n,3,c,c].  Checks the status word and the guard bands."""
    import torch

    n = len(images)
    packed, table = pb.preba_pack(images)
    nb = packed.nbytes
    itemsize = 4 if out_dtype == pb.F32 else 2
    ob = n * 3 * c * c * itemsize
    dev = torch.device("cuda:0")
    pix_buf = torch.full((GUARD + nb + GUARD,), CANARY, dtype=torch.uint8, device=dev)
    pix_buf[GUARD:GUARD + nb] = torch.from_numpy(packed).to(dev)
    out_buf = torch.full((GUARD + ob + GUARD,), CANARY, dtype=torch.uint8, device=dev)
    tab = torch.from_numpy(table.view(np.uint8)).to(dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    # dynamic: warps claim slabs through the scratch counters; else fixed shares
    scratch = torch.zeros(pb.SCRATCH_BYTES // 4, dtype=torch.int32, device=dev) if dynamic else None
    pix = pix_buf[GUARD:GUARD + nb]
    out = out_buf[GUARD:GUARD + ob]
    torch.cuda.synchronize()
    pb.preba_preprocess(pix, tab, n, out, c, s, mean, std, out_dtype, stream=stream,
                        table_host=table if check_host_table else None, status=status,
                        scratch=scratch)
    torch.cuda.synchronize()
    assert int(status.item()) == 0, pb.preba_strerror(int(status.item()))
    if scratch is not None:
        assert int(scratch.abs().sum().item()) == 0, "the launch did not leave its scratch zeroed"
    ob_host = out_buf.cpu().numpy()
    assert np.all(ob_host[:GUARD] == CANARY) and np.all(ob_host[GUARD + ob:] == CANARY), \
        "kernel wrote outside the output tensor"
    pb_host = pix_buf.cpu().numpy()
    assert np.all(pb_host[:GUARD] == CANARY) and np.all(pb_host[GUARD + nb:] == CANARY)
    assert np.array_equal(pb_host[GUARD:GUARD + nb], packed), "kernel modified its input"
    res = ob_host[GUARD:GUARD + ob].copy()
    view = {pb.F32: np.float32, pb.F16: np.float16, pb.BF16: np.uint16}[out_dtype]
    return res.view(view).reshape(n, 3, c, c)  # bfloat16 comes back as bit patterns


def oracle_f64(images, c, s, mean=MEAN, std=STD):
    return oracle.preprocess(images, c, s, mean, std, oracle.OUT_F64, nthreads=host_threads())


def _ordered(h16: np.ndarray) -> np.ndarray:
    """Map binary16 bit patterns to integers whose difference is the distance in ulps."""
    b = h16.view(np.uint16).astype(np.int32)
    return np.where(b & 0x8000, -(b & 0x7FFF), b & 0x7FFF)


def fp16_report(gpu_h: np.ndarray, want64: np.ndarray) -> dict:
    """The fp16 criterion: an element passes if it is within one binary16 ulp of the
    double result rounded once to binary16, or if its value is within FP16_ABS of the
    double result.  (Near zero binary16 spacing is far finer than the rounding error of
    fp32 interpolation, so the first clause alone cannot hold there.)"""
    with np.errstate(over="ignore"):
        want_h = want64.astype(np.float16)
    ulps = np.abs(_ordered(gpu_h) - _ordered(want_h))
    abs_err = np.abs(gpu_h.astype(np.float64) - want64)
    strict = ulps <= 1
    ok = strict | (abs_err <= FP16_ABS)
    return dict(failures=int((~ok).sum()), needed_abs_clause=int((~strict & ok).sum()),
                max_ulps=int(ulps.max()), exact=int((ulps == 0).sum()), total=int(ulps.size),
                max_abs_err=float(abs_err.max()))


def bf16_bits_to_float(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << 16).view(np.float32)


def bf16_report(gpu_bits: np.ndarray, want64: np.ndarray) -> dict:
    """The fp16 criterion carried over to bfloat16: within one bfloat16 ulp of the double
    result rounded once (by the oracle's own rounding routine), or within FP16_ABS of it."""
    flat = want64.reshape(-1)
    want_bits = np.fromiter((oracle.round_bf16_bits(v) for v in flat), dtype=np.uint16,
                            count=flat.size).reshape(want64.shape)
    ulps = np.abs(_ordered(gpu_bits) - _ordered(want_bits))
    abs_err = np.abs(bf16_bits_to_float(gpu_bits).astype(np.float64) - want64)
    strict = ulps <= 1
    ok = strict | (abs_err <= FP16_ABS)
    return dict(failures=int((~ok).sum()), needed_abs_clause=int((~strict & ok).sum()),
                max_ulps=int(ulps.max()), exact=int((ulps == 0).sum()), total=int(ulps.size))


def assert_parity(gpu: np.ndarray, want64: np.ndarray, out_dtype: int) -> dict:
    assert gpu.shape == want64.shape
    if out_dtype == pb.BF16:
        rep = bf16_report(gpu, want64)
        assert rep["failures"] == 0, rep
        return rep
    if out_dtype == pb.F32:
        err = float(np.max(np.abs(gpu.astype(np.float64) - want64)))
        assert err <= FP32_TOL, f"fp32 max abs error {err:.3e} > {FP32_TOL}"
        return dict(max_abs_err=err)
    rep = fp16_report(gpu, want64)
    assert rep["failures"] == 0, rep
    return rep
