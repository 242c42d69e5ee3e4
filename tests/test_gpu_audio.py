"""GPU parity of the audio path (log Mel spectrogram, three-pass normalisation) against the
float64 oracle, through the C ABI; host-side checks of sizes, packing and arguments."""
from __future__ import annotations

import ctypes

import numpy as np
import pytest

from oracle import audio as oa
from paper_2411_19114_b200 import binding as pb
from paper_2411_19114_b200 import workloads as wl

# fp32 FFT of 512 points, fp32 Mel sums and logf against float64.  The transform's error is
# about 9 roundings (3 radix-8 passes) relative to the norm of the frame's spectrum, 9 * 2^-24 =
# 5e-7; the weakest Mel band of the test signals lies about 45 dB (3e4 in power, 180 in
# amplitude) below the strongest, so its energy carries a relative error up to about
# 2 * 180 * 5e-7 = 2e-4 in the worst case and about 1e-4 typically, which the log turns into
# the same absolute error (measured 1.2e-4 and 8.6e-5).  The tests allow three times the
# typical figure.
LOGMEL_TOL = 3e-4
NORM_TOL = 3e-4


def test_sizes_and_pack_layout():
    rng = np.random.default_rng(1)
    utts = [rng.uniform(-1, 1, size=n).astype(np.float32) for n in (401, 0, 399, 1601, 16000)]
    s = pb.preba_audio_query([u.size for u in utts])
    offs, at = [], 0
    for u in utts:
        offs.append(at)
        at = -(-(at + u.size) // 4) * 4
    assert s.packed_samples == at and s.table_bytes == 16 * 5
    assert s.t_max == oa.num_frames(16000) == 98 and s.out_bytes == 5 * 80 * 98 * 4
    packed, table = pb.preba_audio_pack(utts)
    assert [int(e["offset"]) for e in table] == offs
    assert [int(e["frames"]) for e in table] == [oa.num_frames(u.size) for u in utts]
    covered = np.zeros(at, dtype=bool)
    for u, o in zip(utts, offs):
        assert np.array_equal(packed[o:o + u.size], u)
        covered[o:o + u.size] = True
    assert np.all(packed[~covered] == 0.0)


def test_audio_entry_point_rejects_bad_arguments_before_any_launch():
    L = pb.lib()
    assert L.preba_audio_logmel(None, 1, None) == pb.ERR_INVALID_ARG
    t = np.zeros(1, dtype=pb.UTT_DTYPE)
    t[0] = (0, 800, 3)

    def call(**kw):
        b = pb.PrebaAudioBatch()
        b.samples, b.samples_count = 0x10000, 800
        b.table, b.table_host = 0x20000, t.ctypes.data
        b.n, b.t_max = 1, 3
        b.out, b.out_bytes = 0x30000, 80 * 3 * 4
        for k, v in kw.items():
            setattr(b, k, v)
        return L.preba_audio_logmel(ctypes.byref(b), 1, None)

    assert call(samples=None) == pb.ERR_INVALID_ARG
    assert call(samples=0x10004) == pb.ERR_INVALID_ARG          # misaligned samples
    assert call(n=0) == pb.ERR_INVALID_ARG
    assert call(t_max=0) == pb.ERR_INVALID_ARG
    assert call(out_bytes=80 * 3 * 4 - 1) == pb.ERR_BUFFER_TOO_SMALL
    assert call(samples_count=799) == pb.ERR_BAD_TABLE          # runs past the samples
    assert call(t_max=2, out_bytes=80 * 3 * 4) == pb.ERR_BAD_TABLE  # more frames than the result holds
    t[0] = (0, 800, 4)
    assert call() == pb.ERR_BAD_TABLE                           # frame count does not follow from length
    t[0] = (2, 700, 2)
    assert call() == pb.ERR_BAD_TABLE                           # misaligned offset


def run_audio(utts, normalize):
    import torch

    n = len(utts)
    packed, table = pb.preba_audio_pack(utts)
    t_max = max(1, pb.preba_audio_query([u.size for u in utts]).t_max)
    dev = torch.device("cuda:0")
    smp = torch.from_numpy(packed).to(dev)
    tab = torch.from_numpy(table.view(np.uint8)).to(dev)
    guard = 1024
    buf = torch.full((guard + n * 80 * t_max + guard,), 777.0, dtype=torch.float32, device=dev)
    out = buf[guard:guard + n * 80 * t_max]
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    pb.preba_audio_logmel(smp, tab, n, t_max, out, normalize, table_host=table, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    host = buf.cpu().numpy()
    assert np.all(host[:guard] == 777.0) and np.all(host[guard + n * 80 * t_max:] == 777.0)
    return host[guard:guard + n * 80 * t_max].reshape(n, 80, t_max).copy()


@pytest.mark.gpu
@pytest.mark.parametrize("normalize", [False, True])
def test_ragged_batch_matches_the_oracle(normalize):
    rng = np.random.default_rng(2)
    utts = wl.utterances(6, seed=3, min_s=0.2, max_s=2.5)
    utts += [rng.uniform(-1, 1, size=n).astype(np.float32) for n in (400, 399, 0, 559, 560, 561, 720)]
    utts.append(np.zeros(1000, dtype=np.float32))               # silence: every energy is the guard
    got = run_audio(utts, normalize)
    want = oa.preprocess(utts, normalized=normalize)
    assert got.shape == want.shape
    err = np.abs(got.astype(np.float64) - want)
    assert float(err.max()) <= (NORM_TOL if normalize else LOGMEL_TOL), float(err.max())
    for i, u in enumerate(utts):                                 # padding is exactly zero
        assert np.all(got[i, :, oa.num_frames(u.size):] == 0.0)


@pytest.mark.gpu
def test_pure_tones_and_impulses_on_the_gpu():
    """Closed forms on the device itself: a constant gives (200 c)^2 at bin 0 only through the
    first filter's rising edge (weight 0 at 0 Hz): all-guard energies except leakage; an impulse
    gives a flat spectrum w^2, so every filter's energy is w^2 times the sum of its weights."""
    x = np.zeros(400 + 160, dtype=np.float32)
    x[290] = 1.0                                                # frame 0 position 290, frame 1 position 130
    got = run_audio([x], False)[0]
    w = 0.5 - 0.5 * np.cos(2 * np.pi * np.arange(400) / 400)
    fb_sum = oa.mel_filterbank().sum(axis=1)
    for t, pos in ((0, 290), (1, 130)):
        want = np.log(w[pos] ** 2 * fb_sum + 2.0 ** -24)
        assert np.max(np.abs(got[:, t] - want)) <= 1e-3


@pytest.mark.gpu
def test_full_size_utterances_sampled_rows():
    utts = wl.utterances(8, seed=5)
    got = run_audio(utts, True)
    rng = np.random.default_rng(6)
    for i in rng.choice(len(utts), size=3, replace=False):
        want = oa.preprocess([utts[i]])[0]
        t = want.shape[1]
        assert float(np.max(np.abs(got[i, :, :t] - want))) <= NORM_TOL
        assert np.all(got[i, :, t:] == 0.0)


@pytest.mark.gpu
def test_device_side_table_check_skips_bad_entries():
    import torch

    utts = wl.utterances(3, seed=7, min_s=0.2, max_s=0.6)
    packed, table = pb.preba_audio_pack(utts)
    t_max = int(table["frames"].max())
    bad = table.copy()
    bad[1]["frames"] += 1                                        # does not follow from its length
    dev = torch.device("cuda:0")
    smp = torch.from_numpy(packed).to(dev)
    tab = torch.from_numpy(bad.view(np.uint8)).to(dev)
    out = torch.full((3, 80, t_max), 5.0, dtype=torch.float32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    pb.preba_audio_logmel(smp, tab, 3, t_max, out, True, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == pb.ERR_BAD_TABLE
    host = out.cpu().numpy()
    assert np.all(host[1] == 0.0)                                # refused entry: zeros
    want = oa.preprocess(utts)
    for i in (0, 2):
        assert float(np.max(np.abs(host[i] - want[i, :, :t_max]))) <= NORM_TOL


# ---- Resample ------------------------------------------------------------------------------------------

RESAMPLE_TOL = 2e-5   # fp32 taps and sums of <= 80 products of magnitude <= 1 against float64


def test_resample_sizes_and_layout():
    out = pb.preba_audio_resample_query([48000, 44101, 0, 7], 44100, 16000)
    assert out.tolist() == [oa.resampled_length(v, 44100, 16000) for v in (48000, 44101, 0, 7)]
    t = pb.preba_audio_layout([401, 0, 399, 1601])
    assert [int(e["offset"]) for e in t] == [0, 404, 404, 804]
    assert [int(e["frames"]) for e in t] == [1, 0, 0, 8]
    L = pb.lib()
    one = np.zeros(1, dtype=np.uint32)
    assert L.preba_audio_resample_query(one.ctypes.data_as(ctypes.POINTER(ctypes.c_uint32)), 1, 0, 16000,
                                        one.ctypes.data_as(ctypes.POINTER(ctypes.c_uint32))) \
        == pb.ERR_INVALID_ARG
    # rate pairs whose phase table is too large are refused before any launch
    assert L.preba_audio_resample(0x1000, 16, 0x2000, 0x3000, 16, 0x4000, 1, 8, 15999, 16000, None,
                                  None) == pb.ERR_INVALID_ARG
    assert L.preba_audio_resample(None, 16, 0x2000, 0x3000, 16, 0x4000, 1, 8, 48000, 16000, None,
                                  None) == pb.ERR_INVALID_ARG


def run_resample(utts, rate_in, rate_out=16000):
    import torch

    n = len(utts)
    packed, table_in = pb.preba_audio_pack(utts)
    lens_out = pb.preba_audio_resample_query([u.size for u in utts], rate_in, rate_out)
    table_out = pb.preba_audio_layout(lens_out)
    total_out = int(pb.preba_audio_query(lens_out).packed_samples)
    dev = torch.device("cuda:0")
    guard = 256
    buf = torch.full((guard + max(4, total_out) + guard,), 777.0, dtype=torch.float32, device=dev)
    out = buf[guard:guard + max(4, total_out)]
    smp = torch.from_numpy(packed).to(dev) if packed.size else torch.zeros(4, device=dev)
    tin = torch.from_numpy(table_in.view(np.uint8)).to(dev)
    tout = torch.from_numpy(table_out.view(np.uint8)).to(dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    pb.preba_audio_resample(smp, tin, out, tout, n, int(lens_out.max()), rate_in, rate_out,
                            status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    host = buf.cpu().numpy()
    assert np.all(host[:guard] == 777.0) and np.all(host[guard + max(4, total_out):] == 777.0)
    res = host[guard:guard + total_out]
    got = []
    for e in table_out:
        o, ln = int(e["offset"]), int(e["length"])
        got.append(res[o:o + ln].copy())
        assert np.all(res[o + ln:-(-(o + ln) // 4) * 4] == 0.0)       # alignment padding is zero
    return got, table_out


@pytest.mark.gpu
@pytest.mark.parametrize("rate_in", [48000, 44100, 22050, 8000, 16000, 11025])
def test_resample_matches_the_oracle(rate_in):
    rng = np.random.default_rng(rate_in)
    # the samples' meaning does not matter to the interpolator: speech-like signals generated
    # at 16 kHz are simply taken as rate_in material; one empty utterance
    utts = [wl.utterance(rng, s) for s in (0.31, 0.05, 0.2)] + [np.zeros(0, dtype=np.float32)]
    utts.append(rng.uniform(-1, 1, size=977).astype(np.float32))   # white noise: all frequencies
    utts.append(np.ones(5, dtype=np.float32))                       # shorter than the filter
    got, _ = run_resample(utts, rate_in)
    for u, g in zip(utts, got):
        want = oa.resample(u, rate_in, 16000)
        assert g.shape == want.shape
        if want.size:
            assert float(np.max(np.abs(g - want))) <= RESAMPLE_TOL


@pytest.mark.gpu
def test_resample_then_log_mel_end_to_end():
    """48 kHz utterances through Resample, Mel spectrogram and Normalize on the device against
    the same chain of the oracle."""
    import torch

    rng = np.random.default_rng(9)
    utts = [rng.normal(0, 0.2, size=n).clip(-1, 1).astype(np.float32) for n in (48000 // 2, 30011, 1500)]
    got16, table16 = run_resample(utts, 48000)
    dev = torch.device("cuda:0")
    # feed the resampled batch straight into the spectrogram path (packed as the kernel wrote it)
    packed16, _ = pb.preba_audio_pack(got16)
    t_max = max(1, int(table16["frames"].max()))
    feat = torch.empty((3, 80, t_max), dtype=torch.float32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    pb.preba_audio_logmel(torch.from_numpy(packed16).to(dev),
                          torch.from_numpy(table16.view(np.uint8)).to(dev), 3, t_max, feat, True,
                          table_host=table16, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    want = oa.preprocess([oa.resample(u, 48000, 16000) for u in utts])
    assert float(np.max(np.abs(feat.cpu().numpy().astype(np.float64) - want[:, :, :t_max]))) <= NORM_TOL


@pytest.mark.gpu
def test_steps_marked_as_overlapping_leave_the_same_bits_and_complete_in_order():
    """A chain of steps whose spectrogram kernels start without waiting for the step before
    (each into buffers of its own), then a copy ordered behind them without any device-wide
    wait: every result is what a step alone leaves."""
    import torch

    dev = torch.device("cuda:0")
    utts = wl.utterances(12, seed=901)
    packed, table = pb.preba_audio_pack(utts)
    t_max = int(table["frames"].max())
    n = len(utts)
    smp = torch.from_numpy(packed).to(dev)
    tab = torch.from_numpy(table.view(np.uint8)).to(dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    alone = torch.empty((n, 80, t_max), dtype=torch.float32, device=dev)
    pb.preba_audio_logmel(smp, tab, n, t_max, alone, True, status=status)
    torch.cuda.synchronize()
    stream = torch.cuda.Stream(device=dev)
    outs = [torch.full((n, 80, t_max), float("nan"), dtype=torch.float32, device=dev) for _ in range(5)]
    host = [torch.empty((n, 80, t_max), dtype=torch.float32).pin_memory() for _ in range(5)]
    done = torch.cuda.Event()
    with torch.cuda.stream(stream):
        for i, o in enumerate(outs):
            pb.PreparedAudio(smp, tab, n, t_max, o, True, stream=stream, status=status,
                             overlap_previous=i > 0)()
        for o, h in zip(outs, host):
            h.copy_(o, non_blocking=True)
        done.record(stream)
    done.synchronize()
    assert int(status.item()) == 0
    want = alone.cpu()
    for h in host:
        assert torch.equal(h, want)


def test_unknown_bits_of_the_normalize_argument_are_refused():
    import ctypes

    b = pb.PrebaAudioBatch()
    assert pb.lib().preba_audio_logmel(ctypes.byref(b), 4, None) == pb.ERR_INVALID_ARG
