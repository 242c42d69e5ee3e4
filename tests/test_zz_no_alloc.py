"""The allocation-free host entry point, preba_preprocess_host_noalloc.

It serves callers that cannot obtain device memory (a plug-in inside a server that owns
the allocator, a latency path where cudaMalloc's device-wide synchronisation is not
allowed, a process with a memory budget fixed at start-up): host buffers in, host buffers
out, staged through an array that is part of the library image.  The tests call it through
the C ABI and hold it to the existing host entry point, which stages through
caller-allocated device buffers: same kernel, so the same bits.  This file sorts last, so a
run that stops at the first failure has already been through every other test.
"""
from __future__ import annotations

import ctypes

import numpy as np
import pytest

from paper_2411_19114_b200 import binding as pb
from paper_2411_19114_b200 import build as pbuild
from paper_2411_19114_b200 import workloads as wl

from helpers import MEAN, STD, assert_parity, oracle_f64


@pytest.fixture(scope="module", autouse=True)
def built_library():
    pbuild.build()


def test_refuses_a_batch_larger_than_its_staging_space():
    # 128 images of 320x240 with fp32 output need about 106 MB; the library carries 64 MiB.
    # The refusal comes before any CUDA call, so this runs without a GPU.
    n = 128
    h, w = [240] * n, [320] * n
    sizes = pb.preba_query(h, w, 224, pb.F32)
    assert sizes.packed_bytes + sizes.out_bytes > pb.NOALLOC_MAX_BYTES
    table = np.zeros(n, dtype=pb.TABLE_DTYPE)
    at = 0
    for i in range(n):
        table[i] = (at, 240, 320)
        at += -(-(3 * 240 * 320) // 128) * 128
    m = (ctypes.c_float * 3)(*MEAN)
    s = (ctypes.c_float * 3)(*STD)
    fake_host = ctypes.c_void_p(0x10000)  # never dereferenced: the call is refused first
    rc = pb.lib().preba_preprocess_host_noalloc(fake_host, sizes.packed_bytes, table.ctypes.data, n,
                                                fake_host, sizes.out_bytes, None, 224, 256, m, s,
                                                pb.F32, None)
    assert rc == pb.ERR_TOO_LARGE
    assert "staging" in pb.preba_strerror(rc)
    # a size close to 2^64 must not wrap into something that seems to fit
    one = np.zeros(1, dtype=pb.TABLE_DTYPE)
    one[0] = (0, 8, 8)
    rc = pb.lib().preba_preprocess_host_noalloc(fake_host, (1 << 64) - 100, one.ctypes.data, 1,
                                                fake_host, 3 * 224 * 224 * 4, None, 224, 256, m, s,
                                                pb.F32, None)
    assert rc == pb.ERR_TOO_LARGE
    # the usual argument checks still come first
    rc = pb.lib().preba_preprocess_host_noalloc(None, sizes.packed_bytes, table.ctypes.data, n,
                                                fake_host, sizes.out_bytes, None, 224, 256, m, s,
                                                pb.F32, None)
    assert rc == pb.ERR_INVALID_ARG


@pytest.mark.gpu
def test_two_calls_in_a_row_match_the_allocating_entry_point():
    import torch

    dev = torch.device("cuda:0")
    # two different batches, so that bytes left in the shared array by the first call would
    # show up in the second; the second is smaller and of another output type
    cases = [(wl.mixed_smooth(24, seed=71), pb.F16, torch.float16),
             (wl.uniform_320x240(9, seed=72), pb.F32, torch.float32)]
    for images, dt, tdt in cases:
        n = len(images)
        packed, table = pb.preba_pack(images)
        ph = torch.from_numpy(packed).pin_memory()

        # the existing entry point: device staging allocated by the caller
        want_host = torch.zeros((n, 3, 224, 224), dtype=tdt).pin_memory()
        dp = torch.empty(packed.nbytes, dtype=torch.uint8, device=dev)
        dtab = torch.empty(n * 16, dtype=torch.uint8, device=dev)
        dout = torch.empty((n, 3, 224, 224), dtype=tdt, device=dev)
        pb.preba_preprocess_host(ph, table, n, want_host, dp, dtab, dout, 224, 256, MEAN, STD, dt)

        # the new one: nothing but host buffers
        got_host = torch.full((n, 3, 224, 224), float("nan"), dtype=tdt).pin_memory()
        status = torch.full((1,), 99, dtype=torch.int32).pin_memory()
        pb.preba_preprocess_host_noalloc(ph, table, n, got_host, 224, 256, MEAN, STD, dt,
                                         status_host=status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        got, want = got_host.numpy(), want_host.numpy()
        bits = np.uint16 if dt == pb.F16 else np.uint32
        assert np.array_equal(got.view(bits), want.view(bits))
        assert_parity(got, oracle_f64(images, 224, 256), dt)
