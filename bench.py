#!/usr/bin/env python
"""Benchmark of the fused preprocessing path.

A step is one pass of the path over one ragged batch: 256 images, H and W uniform in
[240, 500], smooth-noise content, resize 256 / crop 224 / normalise, fp16 NCHW output.
`value` is images/s with the packed batch already in device memory (one kernel launch per
step); `e2e` is images/s from separate decoded host images: pack into pinned memory, copy
in, kernel, copy the result out.  Prints one JSON line (rank 0).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--workload mixed|320x240|1080p|sweep|streams] [--batch N]
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import sys
import threading
import time
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))

from paper_2411_19114_b200 import accounting  # noqa: E402
from paper_2411_19114_b200 import workloads as wl  # noqa: E402

METRIC = "preprocessed images/sec"
UNIT = "images/s"
FALLBACK_HBM_GBS = 6650.0

# DRAM bytes (read + write) per launch of the kernel on the default workload in steady state:
# the sum over consecutive launches of the rotating-buffer loop, captured by ncu in one pass
# without cache flushes between launches, divided by the launch count (so the write-back of a
# launch's result, which happens while later launches run, is inside the window).  Valid only
# for the kernel sources with this digest (else reported as null).
NCU_TRAFFIC = {"csrc_sha1": "81497e8b38d1e1376b16577b2c748b1bd37ec458", "bytes_per_launch": 75668384 + 76500544}
TRAFFIC_NOTE = ("dram read + write bytes summed over 8 consecutive launches of this loop (one "
                "ncu pass, caches not flushed between launches) / 8")


# The same for the antialiased kernel: captured on 32 frames of 1080 x 1920 (traffic grows in
# proportion to the frames, so a launch over n frames is taken as n / 32 of it).
AA_NCU_TRAFFIC = {"csrc_sha1": "55e9f17f9e819ba125b9eb1d2077e366cb9c484e", "frames": 32,
                  "bytes": 90032640 + 7090944}


def csrc_digest(name: str = "preba_kernels.cu") -> str:
    """SHA-1 of the source file that holds a kernel and its launch code."""
    path = ROOT / "paper_2411_19114_b200" / "csrc" / name
    return hashlib.sha1(path.read_bytes()).hexdigest()


def make_workload(name: str, batch: int | None, rank: int):
    """(images, out dtype name, description).  Every rank draws its own batch."""
    shift = 1000 * rank
    if name == "mixed":
        n = batch or 256
        return wl.mixed_smooth(n, seed=2 + shift), "f16", \
            f"{n} mixed-size images, H,W~U[240,500], smooth noise, fp16 out (ragged batch)"
    if name == "320x240":
        n = batch or 64
        return wl.uniform_320x240(n, seed=1 + shift), "f32", \
            f"{n} images 320x240, uniform bytes, fp32 out"
    if name == "1080p":
        n = batch or 64
        return wl.hires_1080p(n, seed=4 + shift), "f32", \
            f"{n} images 1920x1080, smooth noise, fp32 out"
    if name == "streams":
        n = batch or 32
        return wl.server_batch_500x375(0, n), "f16", \
            f"{n} images 500x375, smooth noise, fp16 out (one of 7 servers)"
    if name == "sweep":
        n = batch or 2048
        return wl.sweep_500x375(n, seed=5 + shift), "f16", \
            f"{n} images 500x375, uniform bytes, fp16 out"
    raise SystemExit(f"unknown workload {name}")


def config_of(desc: str, dtype: str, n: int, world: int) -> dict:
    """The workload description both arms report."""
    return {"workload": desc, "resize_short": wl.RESIZE_SHORT, "out_size": wl.OUT_SIZE,
            "out_dtype": dtype, "images_per_step_per_gpu": n,
            "parallelism": f"dp{world} (independent batches, no collective)"}


def max_over_ranks(values, dist, device):
    """Element-wise maximum of a list of floats over all ranks (identity without a group)."""
    if dist is None:
        return [float(v) for v in values]
    import torch

    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.tolist()]


def measured_peak() -> tuple[float, str]:
    p = ROOT / "MEASURED_PEAKS.json"
    try:
        return float(json.loads(p.read_text())["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (no MEASURED_PEAKS.json)"


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU through NVML while a region runs."""

    REASONS = {
        0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown",
        0x4: "sw_power_cap", 0x80: "hw_power_brake", 0x2: "applications_clocks_setting",
        0x100: "display_clock_setting", 0x10: "sync_boost",
    }

    def __init__(self, index: int, period_s: float = 0.002):
        self.index, self.period = index, period_s
        self.sm, self.bits, self.max_mhz = [], 0, None
        self._stop = threading.Event()
        self._thread = None
        self._nv = self._dev = None
        self.error = None

    def _open(self):
        """NVML handle of the GPU (by UUID, so that CUDA_VISIBLE_DEVICES does not mislead)."""
        import pynvml as nv

        nv.nvmlInit()
        uuid = None
        try:
            import torch

            uuid = "GPU-" + str(torch.cuda.get_device_properties(self.index).uuid)
        except Exception:
            pass
        try:
            dev = nv.nvmlDeviceGetHandleByUUID(uuid.encode() if uuid else b"")
        except Exception:
            dev = nv.nvmlDeviceGetHandleByIndex(self.index)
        self._nv, self._dev = nv, dev
        self.max_mhz = int(nv.nvmlDeviceGetMaxClockInfo(dev, nv.NVML_CLOCK_SM))

    def sample(self):
        """One reading of the SM clock and the reasons word, taken by the caller."""
        nv, dev = self._nv, self._dev
        if nv is None:
            return
        try:
            self.sm.append(int(nv.nvmlDeviceGetClockInfo(dev, nv.NVML_CLOCK_SM)))
            try:
                self.bits |= int(nv.nvmlDeviceGetCurrentClocksEventReasons(dev))
            except Exception:
                self.bits |= int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(dev))
        except Exception as exc:
            self.error = repr(exc)

    def _run(self):
        while not self._stop.is_set():
            self.sample()
            self._stop.wait(self.period)

    def open(self):
        """Set NVML up ahead of time (before the warm-up), so that entering the timed region
        costs nothing and the first sample is immediate."""
        if self._nv is None and self.error is None:
            try:
                self._open()
            except Exception as exc:  # NVML missing: report, do not invent numbers
                self.error = repr(exc)
        return self

    def __enter__(self):
        self.open()
        if self._nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *a):
        # one reading while the last launches are still in flight or have only just ended
        self.sample()
        self._stop.set()
        if self._thread is not None:
            self._thread.join(timeout=5)

    def summary(self) -> dict:
        if not self.sm:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [],
                    "error": self.error or "no samples"}
        reasons = [name for bit, name in self.REASONS.items() if self.bits & bit]
        return {"sm_mhz": float(np.median(self.sm)), "sm_max_mhz": self.max_mhz,
                "reasons": reasons, "samples": len(self.sm)}


def cpu_threads() -> int:
    return max(1, len(os.sched_getaffinity(0)))


def time_oracle(images, out_kind_name: str, budget_s: float, max_passes: int, threads=None):
    """The oracle as it stands, all host threads (or `threads`), whole batch per pass."""
    import oracle

    kind = oracle.OUT_F16 if out_kind_name == "f16" else oracle.OUT_F32
    packed, offsets, h, w = oracle.pack(images)
    threads = min(threads or cpu_threads(), len(images))
    times = []
    t_end = time.perf_counter() + budget_s
    while len(times) < max_passes:
        t0 = time.perf_counter()
        oracle.preprocess_packed(packed, offsets, h, w, wl.OUT_SIZE, wl.RESIZE_SHORT, wl.MEAN,
                                 wl.STD, kind, nthreads=threads)
        times.append(time.perf_counter() - t0)
        if time.perf_counter() > t_end:
            break
    return times, threads


def run_reference(args, rank: int, world: int) -> None:
    """The reference arm: the CPU oracle on the host cores (rank 0 only)."""
    if rank != 0:
        return
    images, dtype, desc = make_workload(args.workload, args.batch, 0)
    n = len(images)
    warm, _ = time_oracle(images, dtype, 30.0, max(1, args.warmup))
    times, threads = time_oracle(images, dtype, 60.0, max(1, args.steps))
    total = float(sum(times))
    value = n * len(times) / total
    sample = (f"whole batch of {n} images per step, {len(times)} steps after {len(warm)} warm-up "
              "steps (time budgets 60 s and 30 s)")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": len(times), "warmup": len(warm), "ms_per_step": 1e3 * total / len(times),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": config_of(desc, dtype, n, max(1, args.gpus)),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def run_streams(args, local_rank: int) -> None:
    """Seven small inference servers sharing one GPU (the paper's 1g.5gb x 7 set-up, Sec. 3):
    seven streams, each with its own batch of 32 images of 500x375, batch after batch;
    reports aggregate images/s and per-batch latency percentiles."""
    import torch

    from paper_2411_19114_b200 import binding as pb

    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device (the CUDA path has no CPU fallback)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    pb.lib()
    n_streams, n, C, S = 7, args.batch or 32, wl.OUT_SIZE, wl.RESIZE_SHORT
    steps, warm = args.steps, max(args.warmup, 3)
    ctx = []
    acct_total = 0
    for sidx in range(n_streams):
        images = wl.server_batch_500x375(sidx, n)
        packed, table = pb.preba_pack(images)
        acct_total += accounting.batch_bytes(table, C, S, 2)["total"]
        st = torch.cuda.Stream(device=dev)
        pix = torch.from_numpy(packed).to(dev)
        tab = torch.from_numpy(table.view(np.uint8)).to(dev)
        out = torch.empty((n, 3, C, C), dtype=torch.float16, device=dev)
        status = torch.zeros(1, dtype=torch.int32, device=dev)
        call = pb.PreparedPreprocess(pix, tab, n, out, C, S, wl.MEAN, wl.STD, pb.F16, stream=st,
                                     status=status)
        # the same batch alone on the default stream: the concurrent run must give these bits
        alone = torch.empty_like(out)
        pb.preba_preprocess(pix, tab, n, alone, C, S, wl.MEAN, wl.STD, pb.F16, status=status)
        ctx.append(dict(stream=st, call=call, out=out, alone=alone, status=status, keep=(pix, tab)))
    torch.cuda.synchronize()
    # Seven host threads, one per stream; each runs its launch loop inside the library
    # (preba_preprocess_repeated: every launch bracketed by events), so the threads do not
    # queue for the interpreter lock.
    gate = threading.Barrier(n_streams)
    lat = [None] * n_streams
    span = [None] * n_streams
    errors = []

    def server(sidx):
        try:
            call = ctx[sidx]["call"]
            call.repeated(warm)
            gate.wait()
            lat[sidx], span[sidx] = call.repeated(steps)
        except Exception as exc:  # surfaced after the join
            errors.append(exc)
            gate.abort()

    with ClockSampler(local_rank) as clocks:
        threads = [threading.Thread(target=server, args=(i,)) for i in range(n_streams)]
        for t in threads:
            t.start()
        for t in threads:
            t.join()
    if errors:
        raise errors[0]
    torch.cuda.synchronize()
    same = all(int(c["status"].item()) == 0 and bool(torch.equal(c["out"], c["alone"])) for c in ctx)
    assert same, "concurrent streams changed the result"
    elapsed_ms = max(span)
    peak, peak_src = measured_peak()
    achieved = acct_total * steps / (elapsed_ms * 1e-3) / 1e9
    all_lat = np.concatenate(lat)
    line = {
        "metric": METRIC, "value": n_streams * n * steps / (elapsed_ms * 1e-3), "unit": UNIT,
        "n_gpus": 1, "steps": steps, "warmup": warm, "ms_per_step": elapsed_ms / steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic",
        "config": config_of(f"{n_streams} concurrent streams x {n} images 500x375, smooth "
                            "noise, fp16 out", "f16", n, 1),
        "launch": "7 host threads, one stream each, launch loops inside the library",
        "l2": "inputs and outputs of all streams stay resident (warm L2)",
        "streams": {"count": n_streams,
                    "batch_latency_us": {"p50": float(np.percentile(all_lat, 50)),
                                         "p95": float(np.percentile(all_lat, 95)),
                                         "p99": float(np.percentile(all_lat, 99))},
                    "per_stream_p99_us": [float(np.percentile(v, 99)) for v in lat],
                    "bits_identical_to_serial": same},
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "traffic": None, "peak_source": peak_src,
                     "algorithmic_bytes_per_launch": acct_total // n_streams},
        "gpu_launches": n_streams * steps, "clocks": clocks.summary(),
    }
    print(json.dumps(line), flush=True)


# Algorithmic fp32 operations of the audio path per frame: window 400, real 512-point FFT
# 2.5 N log2 N = 11520, power spectrum 3 x 257, Mel filters 2 per non-zero weight (510),
# log 80, three-pass normalisation 6 x 80.
AUDIO_FLOPS_PER_FRAME = 400 + 11520 + 3 * 257 + 2 * 510 + 80 + 6 * 80
# fp32 multiply-add peak from unit counts and the clock: SMs x 128 lanes x 2 x max SM clock
AUDIO_ALU_PEAK_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12


def run_audio(args, local_rank: int) -> None:
    """The paper's second path (Table 1 "Mel spectrogram" + "Normalize") on a ragged batch of
    synthetic utterances: device-resident throughput, end to end from pinned host samples, and
    the numpy oracle timed on the host."""
    import torch

    from oracle import audio as oa
    from paper_2411_19114_b200 import binding as pb

    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device (the CUDA path has no CPU fallback)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    pb.lib()
    n = args.batch or 64
    utts = wl.utterances(n, seed=11)
    packed, table = pb.preba_audio_pack(utts)
    t_max = int(table["frames"].max())
    frames = int(table["frames"].sum())
    seconds = sum(u.size for u in utts) / wl.AUDIO_RATE
    steps, warm = min(args.steps, 2000), max(args.warmup, 3)
    l2 = torch.cuda.get_device_properties(dev).L2_cache_size
    step_bytes = packed.nbytes + n * 80 * t_max * 4
    sets = max(2, min(32, -(-4 * l2 // step_bytes)))
    smp = [torch.from_numpy(packed).to(dev) for _ in range(sets)]
    outs = [torch.empty((n, 80, t_max), dtype=torch.float32, device=dev) for _ in range(sets)]
    tab = torch.from_numpy(table.view(np.uint8)).to(dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    stream = torch.cuda.current_stream()
    # Every step but the one into buffer set 0 is marked as overlapping: its spectrogram kernel
    # moves in while the Normalize kernel of the step before still runs.  A marked launch may
    # run beside everything back to the last unmarked one, so the step that comes round to set 0
    # again is not marked and no two steps that could overlap share a buffer.
    calls = [pb.PreparedAudio(smp[i], tab, n, t_max, outs[i], True, stream=stream, status=status,
                              overlap_previous=i > 0) for i in range(sets)]
    for i in range(warm):
        calls[i % sets]()
    torch.cuda.synchronize()
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(local_rank) as clocks:
        torch.cuda.synchronize()
        start.record(stream)
        for i in range(warm, warm + steps):      # the rotation goes on where the warm-up ended
            calls[i % sets]()
        stop.record(stream)
        torch.cuda.synchronize()
    ms = start.elapsed_time(stop)
    assert int(status.item()) == 0
    # every buffer set that was written must hold what a step running alone leaves
    alone = torch.empty_like(outs[0])
    pb.PreparedAudio(smp[0], tab, n, t_max, alone, True, stream=stream, status=status)()
    torch.cuda.synchronize()
    written = min(sets, warm + steps)
    assert all(bool(torch.equal(o, alone)) for o in outs[:written]), \
        "overlapped steps changed the result"
    # parity of what was timed, on a sample of utterances
    got = outs[0].cpu().numpy()
    for i in (0, n // 2, n - 1):
        want = oa.preprocess([utts[i]])[0]
        err = float(np.max(np.abs(got[i, :, :want.shape[1]] - want)))
        assert err <= 3e-4, f"audio result differs from the oracle: {err:.3e}"
    # the Resample unit on the same samples taken as 48 kHz material (48 kHz -> 16 kHz)
    lens48 = pb.preba_audio_resample_query(table["length"], 48000, 16000)
    table48 = pb.preba_audio_layout(lens48)
    out48 = torch.empty(int(pb.preba_audio_query(lens48).packed_samples), dtype=torch.float32,
                        device=dev)
    tab48 = torch.from_numpy(table48.view(np.uint8)).to(dev)
    for _ in range(3):
        pb.preba_audio_resample(smp[0], tab, out48, tab48, n, int(lens48.max()), 48000, 16000,
                                status=status)
    torch.cuda.synchronize()
    r_start, r_stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    r_steps = 200
    r_start.record(stream)
    for i in range(r_steps):
        pb.preba_audio_resample(smp[i % sets], tab, out48, tab48, n, int(lens48.max()), 48000,
                                16000, status=status)
    r_stop.record(stream)
    torch.cuda.synchronize()
    resample_us = r_start.elapsed_time(r_stop) / r_steps * 1e3
    assert int(status.item()) == 0
    got48 = out48.cpu().numpy()
    k48 = int(np.argmin(table["length"]))
    want48 = oa.resample(utts[k48], 48000, 16000)
    o48 = int(table48["offset"][k48])
    err48 = float(np.max(np.abs(got48[o48:o48 + want48.size] - want48)))
    assert err48 <= 2e-5, f"resampled audio differs from the oracle: {err48:.3e}"
    # end to end: pinned samples -> device, two kernels, result -> pinned memory
    e2e_steps = max(3, min(args.e2e_steps, steps))
    ph = torch.from_numpy(packed).pin_memory()
    oh = [torch.empty((n, 80, t_max), dtype=torch.float32).pin_memory() for _ in range(2)]
    side = [torch.cuda.Stream(device=dev) for _ in range(2)]
    done = [torch.cuda.Event() for _ in range(2)]
    e_calls = [pb.PreparedAudio(smp[b], tab, n, t_max, outs[b], True, stream=side[b],
                                status=status) for b in range(2)]

    def e2e_step(i):
        b = i % 2
        done[b].synchronize()
        with torch.cuda.stream(side[b]):
            smp[b].copy_(ph, non_blocking=True)
            e_calls[b]()
            oh[b].copy_(outs[b], non_blocking=True)
        done[b].record(side[b])

    for i in range(2):
        e2e_step(i)
    torch.cuda.synchronize()
    e_start, e_stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e_start.record(stream)
    for st in side:
        st.wait_stream(stream)
    for i in range(e2e_steps):
        e2e_step(i)
    for st in side:
        stream.wait_stream(st)
    e_stop.record(stream)
    torch.cuda.synchronize()
    e2e_ms = e_start.elapsed_time(e_stop)
    # the oracle as it stands (numpy, one thread), on a sample of the batch
    t_end, done_frames, spent, k = time.perf_counter() + args.cpu_budget, 0, 0.0, 0
    while k < n and (k == 0 or time.perf_counter() < t_end):
        t0 = time.perf_counter()
        oa.preprocess([utts[k]])
        spent += time.perf_counter() - t0
        done_frames += int(table["frames"][k])
        k += 1
    per_launch_s = ms * 1e-3 / steps
    achieved = frames * AUDIO_FLOPS_PER_FRAME / per_launch_s / 1e12
    line = {
        "metric": "log-Mel frames/sec (audio path)", "value": frames / per_launch_s,
        "unit": "frames/s", "n_gpus": 1, "steps": steps, "warmup": warm,
        "ms_per_step": ms / steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": f"{n} synthetic utterances, 1.5-15 s at 16 kHz ({seconds:.0f} s of "
                               f"audio, {frames} frames of 400 samples every 160), 80 log-Mel "
                               "features, per-utterance normalisation, fp32 out",
                   "utterances_per_step": n, "audio_seconds_per_step": seconds},
        "launch": "two kernels per step (spectrogram, normalise), one stream; every step but the one into buffer set 0 marked as overlapping the step before (programmatic dependent launch)",
        "l2": f"rotating {sets} buffer sets ({sets * step_bytes / 1e6:.0f} MB) > L2 "
              f"({l2 / 1e6:.0f} MB)",
        "roofline": {"bound": "alu", "achieved": achieved, "peak": AUDIO_ALU_PEAK_TFLOPS,
                     "unit": "TFLOP/s", "frac": achieved / AUDIO_ALU_PEAK_TFLOPS, "traffic": None,
                     "peak_source": "148 SMs x 128 fp32 lanes x 2 x 1.965 GHz",
                     "algorithmic_flops_per_frame": AUDIO_FLOPS_PER_FRAME,
                     "kernel_us": per_launch_s * 1e6},
        "cpu_baseline": {"value": done_frames / spent, "unit": "frames/s", "cores": 1,
                         "kind": "oracle", "sample": f"{k} of the {n} utterances, one pass"},
        "e2e": {"value": frames * e2e_steps / (e2e_ms * 1e-3), "unit": "frames/s",
                "h2d_bytes_per_step": int(packed.nbytes), "d2h_bytes_per_step": n * 80 * t_max * 4,
                "steps": e2e_steps, "ms_per_step": e2e_ms / e2e_steps,
                "includes": "packed samples pinned -> device, both kernels, result -> pinned "
                            "memory; two buffer sets on two streams"},
        "audio_seconds_per_second": seconds / per_launch_s,
        "resample_48k_to_16k": {"us_per_launch": resample_us,
                                "input_samples_per_s": float(table["length"].sum()) /
                                                       (resample_us * 1e-6),
                                "note": "the same packed samples taken as 48 kHz material, one "
                                        "kernel per batch; checked against the oracle on the "
                                        "shortest utterance"},
        "gpu_launches": 2 * steps, "clocks": clocks.summary(),
    }
    print(json.dumps(line), flush=True)


def run_antialias(args, local_rank: int) -> None:
    """The antialiased Resize variant on the heavy-reduction batch (64 frames of 1080 x 1920 ->
    224 x 224, fp32): device-resident throughput against the HBM roofline of its footprint,
    end to end from a pinned packed buffer, and its numpy oracle timed on the host."""
    import torch

    from oracle import antialias as oaa
    from paper_2411_19114_b200 import accounting
    from paper_2411_19114_b200 import binding as pb

    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device (the CUDA path has no CPU fallback)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    pb.lib()
    n = args.batch or 64
    images = wl.hires_1080p(n)
    packed, table = pb.preba_pack(images)
    acct = accounting.antialias_batch_bytes(table, wl.OUT_SIZE, wl.RESIZE_SHORT, 4)
    steps, warm = min(args.steps, 500), max(args.warmup, 3)
    l2 = torch.cuda.get_device_properties(dev).L2_cache_size
    sets = 2 if acct["total"] > 2 * l2 else max(2, min(16, -(-4 * l2 // acct["total"])))
    pix = [torch.from_numpy(packed).to(dev) for _ in range(sets)]
    outs = [torch.empty((n, 3, wl.OUT_SIZE, wl.OUT_SIZE), dtype=torch.float32, device=dev)
            for _ in range(sets)]
    tab = torch.from_numpy(table.view(np.uint8)).to(dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    stream = torch.cuda.current_stream()
    calls = [pb.PreparedPreprocessEx(pix[i], tab, n, outs[i], wl.OUT_SIZE, wl.RESIZE_SHORT, wl.MEAN, wl.STD,
                                     pb.F32, stream=stream, table_host=table, status=status,
                                     entry="preba_preprocess_antialias") for i in range(sets)]
    for i in range(warm):
        calls[i % sets]()
    torch.cuda.synchronize()
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(local_rank) as clocks:
        torch.cuda.synchronize()
        start.record(stream)
        for i in range(steps):
            calls[i % sets]()
        stop.record(stream)
        torch.cuda.synchronize()
    ms = start.elapsed_time(stop)
    if int(status.item()) != 0:
        raise SystemExit(f"bench.py: kernel status {int(status.item())}")
    per_launch_s = ms * 1e-3 / steps
    # the plain transform on the same batch, for scale
    plain = pb.PreparedPreprocess(pix[0], tab, n, outs[0], wl.OUT_SIZE, wl.RESIZE_SHORT, wl.MEAN, wl.STD,
                                  pb.F32, stream=stream, table_host=table, status=status)
    for _ in range(3):
        plain()
    torch.cuda.synchronize()
    start.record(stream)
    for _ in range(200):
        plain()
    stop.record(stream)
    torch.cuda.synchronize()
    plain_us = start.elapsed_time(stop) * 1000.0 / 200
    # end to end: pinned packed pixels -> device, kernel, result -> pinned memory
    e2e_steps = max(3, min(args.e2e_steps, 10))
    ph = torch.from_numpy(packed).pin_memory()
    oh = torch.empty((n, 3, wl.OUT_SIZE, wl.OUT_SIZE), dtype=torch.float32).pin_memory()

    def e2e_step():
        pix[0].copy_(ph, non_blocking=True)
        calls[0]()
        oh.copy_(outs[0], non_blocking=True)

    e2e_step()
    torch.cuda.synchronize()
    start.record(stream)
    for _ in range(e2e_steps):
        e2e_step()
    stop.record(stream)
    torch.cuda.synchronize()
    e2e_ms = start.elapsed_time(stop)
    # parity on the spot: the first image of the last set against the oracle
    want = oaa.preprocess(images[:1], wl.OUT_SIZE, wl.RESIZE_SHORT, wl.MEAN, wl.STD)[0]
    err = float(np.max(np.abs(outs[0][0].cpu().numpy() - want)))
    if err > 1e-5:
        raise SystemExit(f"bench.py: antialiased output differs from the oracle by {err:.3g}")
    # the oracle as it stands (numpy), on a sample of the batch
    t_end, done, spent = time.perf_counter() + args.cpu_budget, 0, 0.0
    while done < n and (done == 0 or time.perf_counter() < t_end):
        t0 = time.perf_counter()
        oaa.preprocess(images[done:done + 1], wl.OUT_SIZE, wl.RESIZE_SHORT, wl.MEAN, wl.STD)
        spent += time.perf_counter() - t0
        done += 1
    peak, peak_source = measured_peak()
    achieved = acct["total"] / per_launch_s / 1e9
    traffic = AA_NCU_TRAFFIC["bytes"] * n // AA_NCU_TRAFFIC["frames"] \
        if AA_NCU_TRAFFIC["csrc_sha1"] == csrc_digest("preba_antialias.cu") else None
    line = {
        "metric": "preprocessed images/sec (antialiased Resize)", "value": n / per_launch_s,
        "unit": "images/s", "n_gpus": 1, "steps": steps, "warmup": warm,
        "ms_per_step": ms / steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": f"{n} frames of 1080 x 1920, smooth noise, antialiased resize to "
                               "256 on the shorter side (triangle filter, reduction 4.2), centre "
                               "crop 224, fp32 out",
                   "resize_short": wl.RESIZE_SHORT, "out_size": wl.OUT_SIZE, "images_per_step_per_gpu": n},
        "launch": "one kernel per step, one stream",
        "l2": f"{sets} buffer sets of {acct['total'] / 1e6:.0f} MB touched each > L2 "
              f"({l2 / 1e6:.0f} MB)",
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "traffic": traffic, "peak_source": peak_source,
                     "algorithmic_bytes_per_launch": acct["total"],
                     "input_bytes": acct["input_bytes"], "output_bytes": acct["output_bytes"],
                     "kernel_us": per_launch_s * 1e6},
        "cpu_baseline": {"value": done / spent, "unit": "images/s", "cores": cpu_threads(),
                         "kind": "oracle",
                         "sample": f"{done} of the {n} images, one pass (numpy, its BLAS threads)"},
        "e2e": {"value": n * e2e_steps / (e2e_ms * 1e-3), "unit": "images/s",
                "h2d_bytes_per_step": int(packed.nbytes), "d2h_bytes_per_step": int(oh.numel() * 4),
                "steps": e2e_steps, "ms_per_step": e2e_ms / e2e_steps,
                "includes": "packed pixels pinned -> device (whole frames), kernel, result -> "
                            "pinned memory; one stream"},
        "plain_transform_us": plain_us, "max_abs_err_vs_oracle": err,
        "gpu_launches": steps, "clocks": clocks.summary(),
    }
    print(json.dumps(line), flush=True)


def run_serve(args, local_rank: int) -> None:
    """The front-end under load (paper Sec. 5 "Input query modeling", Sec. 4.3, Sec. 3): single
    images arrive by a seeded Poisson process, wait in the batching queue and leave as batches
    to seven servers sharing the GPU, each running preba_preprocess_images (images read in place
    from pinned memory) on a stream of its own; preba_serve_run drives it in real time.  The
    queue's hyper-parameters come from a profile taken first, as the paper prescribes:
    Batch_max = the batch size at the knee of the throughput curve, Time_queue = the latency
    there divided by the number of servers."""
    import torch

    from paper_2411_19114_b200 import binding as pb

    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device (the CUDA path has no CPU fallback)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    pb.lib()
    C, S, n_servers = wl.OUT_SIZE, wl.RESIZE_SHORT, 7
    images = wl.mixed_smooth(256, seed=2)
    page, starts, at = 4096, [], 0
    for im in images:
        starts.append(at)
        at += -(-im.nbytes // page) * page
    arena = torch.empty(at, dtype=torch.uint8).pin_memory()
    pool = []
    for im, st0 in zip(images, starts):
        view = arena[st0:st0 + im.nbytes].view(im.shape)
        view.copy_(torch.from_numpy(im))
        pool.append(view)
    cap = 256

    def staging():
        return dict(table_host=torch.zeros(16 * cap, dtype=torch.uint8).pin_memory(),
                    out_host=torch.empty((cap, 3, C, C), dtype=torch.float16).pin_memory(),
                    dev_table=torch.empty(16 * cap, dtype=torch.uint8, device=dev),
                    dev_out=torch.empty((cap, 3, C, C), dtype=torch.float16, device=dev),
                    dev_status=torch.zeros(1, dtype=torch.int32, device=dev),
                    dev_scratch=torch.zeros(pb.SCRATCH_BYTES // 4, dtype=torch.int32, device=dev),
                    stream=torch.cuda.Stream(device=dev))

    servers = [staging() for _ in range(n_servers)]
    # ---- the profile: latency and throughput of one server's call against the batch size ----
    profile = []
    st = servers[0]
    for b in (1, 2, 4, 8, 16, 32, 64, 128, 256):
        call = pb.PreparedImages(pool[:b], st["table_host"], st["out_host"][:b], None,
                                 st["dev_table"], st["dev_out"], C, S, wl.MEAN, wl.STD, pb.F16,
                                 stream=st["stream"], dev_status=st["dev_status"],
                                 dev_scratch=st["dev_scratch"], in_place=True)
        times = []
        for it in range(13):
            t0 = time.perf_counter()
            call()
            st["stream"].synchronize()
            times.append(time.perf_counter() - t0)
        lat = float(np.median(times[3:]))
        profile.append({"batch": b, "latency_us": 1e6 * lat, "images_per_s": b / lat})
    best = max(p["images_per_s"] for p in profile)
    knee = next(p for p in profile if p["images_per_s"] >= 0.9 * best)
    batch_max, time_queue_ns = pb.preba_batching_params(knee["batch"],
                                                        int(1e3 * knee["latency_us"]), n_servers)
    # ---- offered loads as fractions of what the profile says the path can carry ----------------
    seconds = 0.25 if args.steps >= 1000 else 0.05
    loads = []
    for frac in (0.1, 0.25, 0.5, 0.7, 0.85, 0.95, 1.05):
        rate = frac * best
        n = int(max(200, min(60000, rate * seconds)))
        rng = np.random.default_rng(1000 + int(100 * frac))
        arrivals = np.cumsum(rng.exponential(1e9 / rate, size=n)).astype(np.uint64)
        which = (np.arange(n) % len(pool)).astype(np.uint32)
        with ClockSampler(local_rank) as clocks:
            rec = pb.preba_serve_run(arrivals, which, pool, batch_max, time_queue_ns, servers, C, S,
                                     wl.MEAN, wl.STD, pb.F16, device=local_rank)
        if any(int(sv["dev_status"].item()) != 0 for sv in servers):
            raise SystemExit("bench.py: a kernel reported an error status")
        lat_us = (rec["done_ns"].astype(np.float64) - arrivals.astype(np.float64)) / 1e3
        span_s = (float(rec["done_ns"].max()) - float(arrivals[0])) / 1e9
        loads.append({"offered_images_per_s": rate, "fraction_of_profile": frac, "requests": n,
                      "achieved_images_per_s": n / span_s,
                      "latency_us": {"p50": float(np.percentile(lat_us, 50)),
                                     "p95": float(np.percentile(lat_us, 95)),
                                     "p99": float(np.percentile(lat_us, 99))},
                      "batches": int(len(rec["batch_size"])),
                      "mean_batch": float(rec["batch_size"].mean()),
                      "clocks": clocks.summary()})
    base = loads[0]["latency_us"]["p95"]
    leaves = next((l["offered_images_per_s"] for l in loads if l["latency_us"]["p95"] > 2 * base),
                  None)
    sustained = [l for l in loads if l["latency_us"]["p95"] <= 2 * base]
    top = max(sustained, key=lambda l: l["achieved_images_per_s"])
    line = {
        "metric": "served images/sec under Poisson load (queue + kernel, host to host)",
        "value": top["achieved_images_per_s"], "unit": UNIT, "n_gpus": 1,
        "steps": sum(l["requests"] for l in loads), "warmup": 0,
        "ms_per_step": None, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": "single-image requests, Poisson arrivals, 256 mixed-size images "
                               "H,W~U[240,500] in turn, batching queue, 7 servers on 7 streams, "
                               "fp16 out", "resize_short": S, "out_size": C, "out_dtype": "f16",
                   "servers": n_servers},
        "batching": {"batch_knee": knee["batch"], "time_knee_us": knee["latency_us"],
                     "batch_max": batch_max, "time_queue_us": time_queue_ns / 1e3,
                     "rule": "Batch_max = Batch_knee (smallest profiled batch within 10 % of the "
                             "best throughput), Time_queue = Time_knee / servers"},
        "profile": profile, "loads": loads,
        "p95_leaves_the_knee_at_images_per_s": leaves,
        "note": "value = the highest achieved rate among the loads whose p95 latency stays "
                "within twice the p95 at the lowest load; latency from a request's arrival time "
                "to the host-side completion of its batch (result in pinned host memory)",
        "gpu_launches": sum(l["batches"] for l in loads), "clocks": loads[-1]["clocks"],
    }
    print(json.dumps(line), flush=True)


def jpeg_roofline(compressed: int, decoded: int, decode_ms: float) -> dict:
    """Decode against the memory it has to touch: the compressed bytes in, the pixels out."""
    peak, source = measured_peak()
    alg = compressed + decoded
    achieved = alg / (decode_ms * 1e-3) / 1e9
    return {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
            "frac": achieved / peak, "traffic": None, "peak_source": source,
            "algorithmic_bytes_per_launch": alg, "kernel_us": 1e3 * decode_ms,
            "note": "the three Decode kernels of a step together (device time); Decode is bound "
                    "by the serial Huffman decoding of a restart interval per thread (latency), "
                    "far from any memory or pipe limit; see the launch list under profiles/"}


def run_jpeg(args, local_rank: int) -> None:
    """Decode in front of the transform (the paper's Decode -> Resize -> Crop -> Normalize chain,
    Sec. 4.2, Table 1): 256 mixed-size synthetic images as baseline JPEG streams (quality 90,
    4:2:0, a restart marker per row of MCUs) in host memory; a step is preba_jpeg_decode (header
    parsing and staging on the host, one copy, three kernels) followed by preba_preprocess on
    the buffers it wrote.  Reports images/s of the whole step, of Decode alone, and the oracle
    decoder on the host."""
    import torch

    from oracle import jpeg as oj
    from paper_2411_19114_b200 import binding as pb

    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device (the CUDA path has no CPU fallback)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    pb.lib()
    n = args.batch or 256
    images = wl.mixed_smooth(n, seed=2)
    jpegs = wl.jpeg_streams(images, quality=90, subsampling=2, restart_rows=1)
    comp_bytes = sum(len(j) for j in jpegs)
    h, w, sz = pb.preba_jpeg_query(jpegs)
    C, S = wl.OUT_SIZE, wl.RESIZE_SHORT
    nbuf = 2
    stream = torch.cuda.current_stream()
    bufs = []
    for _ in range(nbuf):
        b = dict(stage_host=torch.zeros(sz.stage_bytes, dtype=torch.uint8).pin_memory(),
                 stage_dev=torch.zeros(sz.stage_bytes, dtype=torch.uint8, device=dev),
                 coef=torch.zeros(sz.coef_bytes // 2, dtype=torch.int16, device=dev),
                 pixels=torch.zeros(sz.packed_bytes, dtype=torch.uint8, device=dev),
                 table=torch.zeros(16 * n, dtype=torch.uint8, device=dev),
                 table_host=torch.zeros(16 * n, dtype=torch.uint8).pin_memory(),
                 out=torch.empty((n, 3, C, C), dtype=torch.float16, device=dev),
                 done=torch.cuda.Event())
        b["status"] = torch.zeros(1, dtype=torch.int32, device=dev)
        b["decode"] = pb.PreparedJpeg(jpegs, b["stage_host"], b["stage_dev"], b["coef"],
                                      b["pixels"], b["table"], b["table_host"], b["status"],
                                      stream=stream)
        b["transform"] = pb.PreparedPreprocess(b["pixels"], b["table"], n, b["out"], C, S, wl.MEAN,
                                               wl.STD, pb.F16, stream=stream, status=b["status"])
        bufs.append(b)

    def step(i, transform=True):
        b = bufs[i % nbuf]
        b["done"].synchronize()          # the staging buffer is free again
        b["decode"]()
        if transform:
            b["transform"]()
        b["done"].record(stream)

    steps, warm = max(3, min(args.steps, 200)), max(3, min(args.warmup, 10))
    results = {}
    for name, transform in (("decode_and_transform", True), ("decode_only", False)):
        for i in range(warm):
            step(i, transform)
        torch.cuda.synchronize()
        start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with ClockSampler(local_rank) as clocks:
            t0 = time.perf_counter()
            start.record(stream)
            for i in range(steps):
                step(i, transform)
            stop.record(stream)
            torch.cuda.synchronize()
            wall = time.perf_counter() - t0
        results[name] = {"images_per_s": n * steps / wall, "ms_per_step": 1e3 * wall / steps,
                         "device_ms_per_step": start.elapsed_time(stop) / steps,
                         "clocks": clocks.summary()}
    for b in bufs:
        if int(b["status"].item()) != 0:
            raise SystemExit(f"bench.py: kernel status {int(b['status'].item())}")
    # parity on the spot: one decoded image and its transform against the oracles
    import oracle

    k = n // 2
    tab = bufs[0]["table_host"].numpy().view(pb.TABLE_DTYPE)
    off = int(tab[k]["offset"])
    got = bufs[0]["pixels"][off:off + 3 * int(h[k]) * int(w[k])].cpu().numpy().reshape(int(h[k]), int(w[k]), 3)
    t0 = time.perf_counter()
    want = oj.decode(jpegs[k])
    cpu_s = time.perf_counter() - t0
    if not np.array_equal(got, want):
        raise SystemExit("bench.py: decoded image differs from the oracle")
    want_t = oracle.preprocess([want], C, S, wl.MEAN, wl.STD, oracle.OUT_F64)[0]
    err = float(np.max(np.abs(bufs[0]["out"][k].float().cpu().numpy() - want_t)))
    if err > 2e-3:
        raise SystemExit(f"bench.py: transformed image differs from the oracle by {err:.3g}")
    done_cpu, spent = 1, cpu_s
    while spent < args.cpu_budget and done_cpu < n:
        t0 = time.perf_counter()
        oj.decode(jpegs[done_cpu])
        spent += time.perf_counter() - t0
        done_cpu += 1
    both = results["decode_and_transform"]
    line = {
        "metric": "decoded and preprocessed images/sec (JPEG streams in host memory)",
        "value": both["images_per_s"], "unit": UNIT, "n_gpus": 1, "steps": steps, "warmup": warm,
        "ms_per_step": both["ms_per_step"], "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "int64 (inverse DCT, colour), f32 (transform)",
        "data": "synthetic",
        "config": {"workload": f"{n} mixed-size images H,W~U[240,500] as baseline JPEG streams "
                               "(quality 90, 4:2:0, restart marker per MCU row), decode, resize "
                               "256 / crop 224 / normalise, fp16 out",
                   "resize_short": S, "out_size": C, "images_per_step_per_gpu": n,
                   "compressed_bytes_per_step": comp_bytes,
                   "decoded_bytes_per_step": int(sz.packed_bytes)},
        "launch": "per step: host header parsing and staging, one copy, three Decode kernels, "
                  "the transform's kernel; one stream, two buffer sets",
        "timing": "wall clock around the loop of steps (host work is part of a step); "
                  "device_ms_per_step from events on the stream",
        "steps_detail": results,
        "roofline": jpeg_roofline(comp_bytes, int(sz.packed_bytes),
                                  results["decode_only"]["device_ms_per_step"]),
        "cpu_baseline": {"value": done_cpu / spent, "unit": UNIT, "cores": 1, "kind": "oracle",
                         "sample": f"{done_cpu} of the {n} streams, decode only (plain Python)"},
        "e2e": {"value": both["images_per_s"], "unit": UNIT,
                "h2d_bytes_per_step": int(sz.stage_bytes + 16 * n), "d2h_bytes_per_step": 0,
                "note": "the step starts from host memory already: the value is end to end up "
                        "to the device-resident result"},
        "gpu_launches": 4 * steps, "clocks": both["clocks"],
    }
    print(json.dumps(line), flush=True)


def report_variant(args, rank, world, n, elapsed_ms, acct, desc, dtype, sets, step_bytes, l2,
                   clocks, dist, dev, t_host, launch_note) -> None:
    """The JSON line of a --variant run: the device-resident leg only."""
    (elapsed_ms,) = max_over_ranks([elapsed_ms], dist, dev)
    if rank == 0:
        peak, peak_src = measured_peak()
        per_launch_s = elapsed_ms * 1e-3 / args.steps
        achieved = acct["total"] / per_launch_s / 1e9
        line = {
            "metric": METRIC, "value": world * n * args.steps / (elapsed_ms * 1e-3), "unit": UNIT,
            "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
            "ms_per_step": elapsed_ms / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "int32" if dtype == "u8" else "int32+f32",
            "data": "synthetic",
            "config": config_of(desc, dtype, n, world),
            "launch": launch_note,
            "l2": f"rotating {sets} input/output buffer sets "
                  f"({sets * step_bytes / 1e6:.0f} MB held, "
                  f"{sets * acct['total'] / 1e6:.0f} MB touched) > L2 ({l2 / 1e6:.0f} MB)",
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                         "frac": achieved / peak, "traffic": None, "peak_source": peak_src,
                         "algorithmic_bytes_per_launch": acct["total"],
                         "input_sector_bytes": acct["input_sector_bytes"],
                         "output_bytes": acct["output_bytes"],
                         "kernel_us": per_launch_s * 1e6,
                         "host_launch_us": 1e6 * t_host / args.steps},
            "gpu_launches": args.steps, "clocks": clocks.summary(),
        }
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def run_ours(args, rank: int, world: int, local_rank: int) -> None:
    import torch

    from paper_2411_19114_b200 import binding as pb

    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device (the CUDA path has no CPU fallback)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist

        dist.init_process_group("nccl", device_id=dev)
    pb.lib()

    images, dtype, desc = make_workload(args.workload, args.batch, rank)
    n = len(images)
    out_dtype = pb.F16 if dtype == "f16" else pb.F32
    tdt = torch.float16 if dtype == "f16" else torch.float32
    C, S = wl.OUT_SIZE, wl.RESIZE_SHORT

    packed, table = pb.preba_pack(images)
    if args.variant == "u8":
        out_dtype, tdt, dtype = pb.U8, torch.uint8, "u8"
        desc += ", rounded uint8 HWC output (preba_preprocess_ex)"
    elif args.variant == "round":
        desc += ", resized pixel rounded to uint8 before normalising (preba_preprocess_ex)"
    acct = accounting.batch_bytes(table, C, S, {"f16": 2, "f32": 4, "u8": 1}[dtype])
    l2 = torch.cuda.get_device_properties(dev).L2_cache_size
    step_bytes = packed.nbytes + acct["output_bytes"]
    # enough buffer sets that the bytes a launch touches (the tapped sectors and the result,
    # which can be far less than the images), summed over the sets, exceed four times L2; and
    # at least 32 (memory allowing), because the launch that reuses the first set is the one
    # that is not marked as overlapping (see below)
    sets = max(2, min(64, -(-4 * l2 // min(step_bytes, acct["total"]))))
    sets = max(sets, min(32, max(4, (24 << 30) // step_bytes)))
    pix0 = torch.from_numpy(packed).to(dev)
    pix = [pix0] + [pix0.clone() for _ in range(sets - 1)]
    out_shape = (n, C, C, 3) if args.variant == "u8" else (n, 3, C, C)
    outs = [torch.empty(out_shape, dtype=tdt, device=dev) for _ in range(sets)]
    tab = torch.from_numpy(table.view(np.uint8)).to(dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    scratch = torch.zeros(pb.SCRATCH_BYTES // 4, dtype=torch.int32, device=dev)
    stream = torch.cuda.current_stream()

    # Timed launches go to one stream, each into the next buffer set and marked independent
    # of the kernels before it, so a launch starts as the previous one's warps retire.  A
    # marked launch may run beside every kernel back to the last unmarked one, so the launch
    # into set 0, where the buffers come round again, is not marked: it waits for everything
    # before it, and no two launches that could overlap ever share a buffer.
    def prepared(i, flags):
        if args.variant == "plain":
            return pb.PreparedPreprocess(pix[i], tab, n, outs[i], C, S, wl.MEAN, wl.STD, out_dtype,
                                         stream=stream, status=status, flags=flags)
        return pb.PreparedPreprocessEx(pix[i], tab, n, outs[i], C, S, wl.MEAN, wl.STD, out_dtype,
                                       round_u8=True, stream=stream, status=status, flags=flags)

    calls = [prepared(i, pb.OVERLAP_PREVIOUS if i else 0) for i in range(sets)]
    launch_note = (f"one stream, back-to-back launches into {sets} rotating buffer sets; every "
                   "launch but the one into set 0 is marked independent of the kernels before it "
                   "(programmatic dependent launch)")

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident throughput: one launch per step -------------------------------------
    sampler = ClockSampler(local_rank).open()   # NVML is set up before the warm-up
    n_warm = max(args.warmup, 3)
    for i in range(n_warm):
        calls[i % sets]()
    barrier()
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with sampler as clocks:
        barrier()
        start.record(stream)
        t_host = time.perf_counter()
        for i in range(n_warm, n_warm + args.steps):  # the rotation goes on where the warm-up ended
            calls[i % sets]()
        t_host = time.perf_counter() - t_host
        stop.record(stream)
        clocks.sample()                          # while the last launches are still running
        barrier()
    elapsed_ms = start.elapsed_time(stop)
    assert int(status.item()) == 0, "kernel reported an error status"
    # every buffer set must hold the result of an isolated launch
    ref = torch.empty_like(outs[0])
    if args.variant == "plain":
        pb.preba_preprocess(pix[0], tab, n, ref, C, S, wl.MEAN, wl.STD, out_dtype, stream=stream,
                            status=status, scratch=scratch)
    else:
        pb.preba_preprocess_ex(pix[0], tab, n, ref, C, S, wl.MEAN, wl.STD, out_dtype,
                               round_u8=True, stream=stream, status=status, scratch=scratch)
    torch.cuda.synchronize()
    written = min(sets, n_warm + args.steps)     # a short run does not reach every set
    assert all(bool(torch.equal(o, ref)) for o in outs[:written]), \
        "overlapped launches changed the result"
    if args.variant != "plain":
        report_variant(args, rank, world, n, elapsed_ms, acct, desc, dtype, sets, step_bytes, l2,
                       clocks, dist, dev, t_host, launch_note)
        return

    # ---- one launch at a time: device time of a launch that runs alone (no overlap flag, so
    # the library cuts a small batch into finer slabs); events around every launch
    alone = pb.PreparedPreprocess(pix[0], tab, n, outs[0], C, S, wl.MEAN, wl.STD, out_dtype,
                                  stream=stream, status=status, scratch=scratch)
    alone.repeated(20)
    lat_us, _ = alone.repeated(max(50, min(args.steps, 1000)))
    assert bool(torch.equal(outs[0], ref)), "an isolated launch changed the result"
    # the same with fixed shares instead of claimed slabs (no scratch)
    fixed = pb.PreparedPreprocess(pix[0], tab, n, outs[0], C, S, wl.MEAN, wl.STD, out_dtype,
                                  stream=stream, status=status)
    fixed.repeated(20)
    lat_fixed_us, _ = fixed.repeated(max(50, min(args.steps, 1000)))
    assert bool(torch.equal(outs[0], ref)), "an isolated launch changed the result"

    # ---- the same launch over and over on one buffer set (whatever fits stays in L2) -----------
    warm_steps = max(3, min(args.steps, 2000))
    for _ in range(3):
        calls[0]()                                  # set 0's call is the unmarked one
    barrier()
    w_start, w_stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    w_start.record(stream)
    for _ in range(warm_steps):
        calls[0]()
    w_stop.record(stream)
    barrier()
    warm_ms = w_start.elapsed_time(w_stop)

    # ---- end to end from host images ----------------------------------------------------------
    # The decoded images wait in pinned host memory, each in a buffer of its own (carved from
    # one arena in reverse order, page-aligned: not the packed layout).  Every step the kernel
    # fetches the rows it taps from there, across the host-device link, and the result is
    # copied back to pinned memory (preba_preprocess_images with PREBA_IMAGES_IN_PLACE); two
    # buffer sets on two streams, so one step's kernel overlaps the other's result copy.
    e2e_steps = max(3, min(args.e2e_steps, args.steps))
    sizes = pb.preba_query(table["h"], table["w"], C, out_dtype)
    nbuf = 2
    page = 4096
    starts, at = [], 0
    for im in reversed(images):
        starts.append(at)
        at += -(-im.nbytes // page) * page
    starts.reverse()
    arena = torch.empty(at, dtype=torch.uint8).pin_memory()
    pinned = []
    for im, st0 in zip(images, starts):
        view = arena[st0:st0 + im.nbytes].view(im.shape)
        view.copy_(torch.from_numpy(im))
        pinned.append(view)
    oh = [torch.empty((n, 3, C, C), dtype=tdt).pin_memory() for _ in range(nbuf)]
    th = [torch.zeros(n * 16, dtype=torch.uint8).pin_memory() for _ in range(nbuf)]
    dtab = [torch.empty(n * 16, dtype=torch.uint8, device=dev) for _ in range(nbuf)]
    done = [torch.cuda.Event() for _ in range(nbuf)]
    side = [torch.cuda.Stream(device=dev) for _ in range(nbuf)]  # one stream per buffer set
    scr = [torch.zeros(pb.SCRATCH_BYTES // 4, dtype=torch.int32, device=dev) for _ in range(nbuf)]
    # both directions in place: the kernel reads the images from, and writes the result to,
    # pinned host memory; a step is the table copy and one kernel
    e2e_calls = [pb.PreparedImages(pinned, th[b], oh[b], None, dtab[b], None, C, S, wl.MEAN,
                                   wl.STD, out_dtype, stream=side[b], dev_status=status,
                                   dev_scratch=scr[b], in_place=True, out_in_place=True)
                 for b in range(nbuf)]
    # the kernel reads in place, the result is copied back by the copy engine
    back_calls = [pb.PreparedImages(pinned, th[b], oh[b], None, dtab[b], outs[b], C, S, wl.MEAN,
                                    wl.STD, out_dtype, stream=side[b], dev_status=status,
                                    dev_scratch=scr[b], in_place=True) for b in range(nbuf)]
    copy_calls = [pb.PreparedImages(pinned, th[b], oh[b], pix[b], dtab[b], outs[b], C, S, wl.MEAN,
                                    wl.STD, out_dtype, stream=side[b], dev_status=status,
                                    dev_scratch=scr[b]) for b in range(nbuf)]

    def e2e_step(i):
        b = i % nbuf
        done[b].synchronize()                       # the set's previous copies have finished
        t0 = time.perf_counter()
        e2e_calls[b]()
        done[b].record(side[b])
        return time.perf_counter() - t0

    def timed_e2e(step, steps):
        for i in range(2):
            step(i)
        barrier()
        e_start, e_stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t_host = 0.0
        e_start.record(stream)
        for st in side:
            st.wait_stream(stream)                  # the timed region starts on both streams
        for i in range(steps):
            t_host += step(i)                       # host time of the calls, waits excluded
        for st in side:
            stream.wait_stream(st)                  # ... and ends when both are done
        e_stop.record(stream)
        barrier()
        return e_start.elapsed_time(e_stop), t_host

    e2e_ms, t_pack = timed_e2e(e2e_step, e2e_steps)
    assert int(status.item()) == 0
    for b in range(nbuf):                           # the host result is the device result
        assert bool(torch.equal(oh[b], ref.cpu())), "end-to-end result differs"

    for b in range(nbuf):
        oh[b].zero_()

    def back_step(i):
        b = i % nbuf
        done[b].synchronize()
        t0 = time.perf_counter()
        back_calls[b]()
        done[b].record(side[b])
        return time.perf_counter() - t0

    back_ms, back_host = timed_e2e(back_step, e2e_steps)
    assert int(status.item()) == 0
    for b in range(nbuf):
        assert bool(torch.equal(oh[b], ref.cpu())), "end-to-end result differs (copy back)"

    # the same with one copy per image to the device instead of reads in place
    def copy_step(i):
        b = i % nbuf
        done[b].synchronize()
        t0 = time.perf_counter()
        copy_calls[b]()
        done[b].record(side[b])
        return time.perf_counter() - t0

    copied_ms, copied_host = timed_e2e(copy_step, e2e_steps)
    assert int(status.item()) == 0

    # the same from a packed host buffer: preba_pack of the images into pinned memory, one
    # copy of the packed buffer, kernel, copy back (reported for comparison)
    ph = [torch.empty(sizes.packed_bytes, dtype=torch.uint8).pin_memory() for _ in range(nbuf)]
    tp = [np.zeros(n, dtype=pb.TABLE_DTYPE) for _ in range(nbuf)]

    def packed_step(i):
        b = i % nbuf
        done[b].synchronize()
        t0 = time.perf_counter()
        pb.preba_pack(images, ph[b].numpy(), tp[b])
        pb.preba_preprocess_host(ph[b], tp[b], n, oh[b], pix[b], dtab[b], outs[b], C, S, wl.MEAN,
                                 wl.STD, out_dtype, stream=side[b], dev_status=status,
                                 dev_scratch=scr[b])
        done[b].record(side[b])
        return time.perf_counter() - t0

    packed_ms, packed_host = timed_e2e(packed_step, e2e_steps)
    assert int(status.item()) == 0

    # what the host-device link gives a plain pinned copy of the packed batch, each way
    link = {}
    big_out = oh[0].view(torch.uint8).reshape(-1)
    for name, dst, src in (("h2d", pix[0], ph[0]), ("d2h", big_out, outs[0].view(torch.uint8).reshape(-1))):
        l_start, l_stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        dst.copy_(src, non_blocking=True)
        barrier()
        l_start.record(stream)
        for _ in range(3):
            dst.copy_(src, non_blocking=True)
        l_stop.record(stream)
        barrier()
        link[name + "_gbs"] = 3 * src.numel() / (l_start.elapsed_time(l_stop) * 1e-3) / 1e9

    # ... and both ways at once (two streams): what the link carries when it is used in both
    # directions, which is what an end-to-end step does
    src_out = outs[0].view(torch.uint8).reshape(-1)
    d_start = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    d_stop = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    barrier()
    for st in side:
        st.wait_stream(stream)
    with torch.cuda.stream(side[0]):
        d_start[0].record(side[0])
        for _ in range(4):
            pix[0].copy_(ph[0], non_blocking=True)
        d_stop[0].record(side[0])
    with torch.cuda.stream(side[1]):
        d_start[1].record(side[1])
        for _ in range(4):
            big_out.copy_(src_out, non_blocking=True)
        d_stop[1].record(side[1])
    barrier()
    link["both_ways_h2d_gbs"] = 4 * ph[0].numel() / (d_start[0].elapsed_time(d_stop[0]) * 1e-3) / 1e9
    link["both_ways_d2h_gbs"] = 4 * src_out.numel() / (d_start[1].elapsed_time(d_stop[1]) * 1e-3) / 1e9

    elapsed_ms, e2e_ms, packed_ms, copied_ms, back_ms = max_over_ranks(
        [elapsed_ms, e2e_ms, packed_ms, copied_ms, back_ms], dist, dev)

    if rank == 0:
        peak, peak_src = measured_peak()
        per_launch_s = elapsed_ms * 1e-3 / args.steps
        achieved = acct["total"] / per_launch_s / 1e9
        traffic = NCU_TRAFFIC["bytes_per_launch"] \
            if NCU_TRAFFIC["csrc_sha1"] == csrc_digest() and args.workload == "mixed" \
            and not args.batch else None
        iso_p50 = float(np.percentile(lat_us, 50))
        cpu_times, threads = time_oracle(images, dtype, args.cpu_budget, 50)
        cpu_value = n * len(cpu_times) / float(sum(cpu_times))
        one_times, _ = time_oracle(images[:max(1, n // 16)], dtype, args.cpu_budget / 4, 5, threads=1)
        cpu_one = max(1, n // 16) * len(one_times) / float(sum(one_times))
        line = {
            "metric": METRIC, "value": world * n * args.steps / (elapsed_ms * 1e-3), "unit": UNIT,
            "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
            "ms_per_step": elapsed_ms / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": config_of(desc, dtype, n, world),
            "launch": launch_note,
            "l2": f"rotating {sets} input/output buffer sets "
                  f"({sets * step_bytes / 1e6:.0f} MB held, "
                  f"{sets * acct['total'] / 1e6:.0f} MB touched) > L2 ({l2 / 1e6:.0f} MB)",
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                         "frac": achieved / peak, "traffic": traffic,
                         "traffic_note": TRAFFIC_NOTE if traffic is not None else None,
                         "peak_source": peak_src,
                         "algorithmic_bytes_per_launch": acct["total"],
                         "input_sector_bytes": acct["input_sector_bytes"],
                         "output_bytes": acct["output_bytes"],
                         "kernel_us": per_launch_s * 1e6,
                         "frac_note": "launches follow one another on the stream and overlap "
                                      "at their ends (see launch); frac_isolated is one launch "
                                      "running alone",
                         "achieved_isolated": acct["total"] / (iso_p50 * 1e-6) / 1e9,
                         "frac_isolated": acct["total"] / (iso_p50 * 1e-6) / 1e9 / peak,
                         "isolated_kernel_us": iso_p50,
                         "host_launch_us": 1e6 * t_host / args.steps},
            "cpu_baseline": {"value": cpu_value, "unit": UNIT, "cores": threads, "kind": "oracle",
                             "sample": f"whole batch of {n} images, {len(cpu_times)} passes",
                             "one_thread_value": cpu_one},
            "e2e": {"value": world * n * e2e_steps / (e2e_ms * 1e-3), "unit": UNIT,
                    "h2d_bytes_per_step": int(acct["input_sector_bytes"] + sizes.table_bytes),
                    "d2h_bytes_per_step": int(sizes.out_bytes), "steps": e2e_steps,
                    "ms_per_step": e2e_ms / e2e_steps,
                    "host_ms_per_step": 1e3 * t_pack / e2e_steps,
                    "link_plain_copy_gbs": link,
                    "achieved_link_gbs": {
                        "h2d": (acct["input_sector_bytes"] + sizes.table_bytes) * e2e_steps
                               / (e2e_ms * 1e-3) / 1e9,
                        "d2h": sizes.out_bytes * e2e_steps / (e2e_ms * 1e-3) / 1e9},
                    "link_bound_ms_per_step": 1e3 * max(
                        (acct["input_sector_bytes"] + sizes.table_bytes)
                        / (link["both_ways_h2d_gbs"] * 1e9),
                        sizes.out_bytes / (link["both_ways_d2h_gbs"] * 1e9)),
                    "link_bound_note": "bytes each way over what a plain pinned copy gets in "
                                       "that direction while the other direction is busy too",
                    "includes": "preba_preprocess_images with both directions in place: the "
                                "kernel fetches the tapped rows of every image from its own "
                                "pinned host buffer across the link and stores the result "
                                "straight into pinned host memory (table copy + one kernel per "
                                "step); two buffer sets on two streams",
                    "h2d_bytes_note": "the tapped sectors and the table: what crosses the link "
                                      f"(the images themselves hold {int(sizes.packed_bytes)} "
                                      "bytes)",
                    "kernel_reads_result_copied_back": {
                        "value": world * n * e2e_steps / (back_ms * 1e-3),
                        "ms_per_step": back_ms / e2e_steps,
                        "host_ms_per_step": 1e3 * back_host / e2e_steps},
                    "one_copy_per_image": {
                        "value": world * n * e2e_steps / (copied_ms * 1e-3),
                        "ms_per_step": copied_ms / e2e_steps,
                        "host_ms_per_step": 1e3 * copied_host / e2e_steps},
                    "from_packed_host_buffer": {
                        "value": world * n * e2e_steps / (packed_ms * 1e-3),
                        "ms_per_step": packed_ms / e2e_steps,
                        "host_ms_per_step": 1e3 * packed_host / e2e_steps,
                        "includes": "preba_pack into pinned memory + one copy + kernel + copy "
                                    "back (preba_preprocess_host)"}},
            "isolated_launch_us": {"p50": iso_p50,
                                   "p99": float(np.percentile(lat_us, 99)),
                                   "fixed_shares_p50": float(np.percentile(lat_fixed_us, 50)),
                                   "note": "device time of one launch running alone (warps claim "
                                           "slabs through the scratch counters; fixed_shares: "
                                           "without scratch), events around every launch, same "
                                           "buffers every time"},
            "warm_l2": {"value": world * n * warm_steps / (warm_ms * 1e-3), "unit": UNIT,
                        "us_per_launch": 1e3 * warm_ms / warm_steps,
                        "note": "one buffer set reused by every launch, launches not marked as "
                                "overlapping; not the headline"},
            "gpu_launches": args.steps,
            "clocks": clocks.summary(),
        }
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def spawn_ranks(n: int) -> int:
    """`--gpus N` without a launcher around it: start the N ranks (one process per GPU) through
    torch.distributed.run on this node, with the same arguments, and pass their output on."""
    import socket
    import subprocess

    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), str(Path(__file__).resolve()),
           *sys.argv[1:]]
    return subprocess.run(cmd).returncode


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=4000)
    ap.add_argument("--warmup", type=int, default=200)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="mixed",
                    choices=["mixed", "320x240", "1080p", "sweep", "streams", "audio", "antialias",
                             "serve", "jpeg"])
    ap.add_argument("--batch", type=int, default=None)
    ap.add_argument("--variant", default="plain", choices=["plain", "u8", "round"],
                    help="device-resident leg through preba_preprocess_ex: u8 = rounded uint8 "
                         "HWC output, round = rounded to uint8 then normalised (workload's dtype)")
    ap.add_argument("--e2e-steps", type=int, default=20)
    ap.add_argument("--cpu-budget", type=float, default=12.0,
                    help="seconds of wall time given to the CPU-baseline leg")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl == "ours" \
            and args.workload in ("mixed", "320x240", "1080p", "sweep"):
        raise SystemExit(spawn_ranks(args.gpus))
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank, world)
    elif args.workload == "streams":
        if rank == 0:
            run_streams(args, local_rank)
    elif args.workload == "audio":
        if rank == 0:
            run_audio(args, local_rank)
    elif args.workload == "antialias":
        if rank == 0:
            run_antialias(args, local_rank)
    elif args.workload == "serve":
        if rank == 0:
            run_serve(args, local_rank)
    elif args.workload == "jpeg":
        if rank == 0:
            run_jpeg(args, local_rank)
    else:
        run_ours(args, rank, world, local_rank)


if __name__ == "__main__":
    main()
