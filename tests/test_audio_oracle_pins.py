"""Pins for the audio oracle (framing, window, spectrum, Mel filters, log, three-pass
normalisation).  Expected values come from closed forms, a direct DFT sum written here,
numpy.interp as an independent triangle, invariants and hand-worked numbers; none from the
function under test."""
from __future__ import annotations

import numpy as np

from oracle import audio as oa


def test_frame_count_closed_form():
    assert [oa.num_frames(n) for n in (0, 399, 400, 559, 560, 720, 16000, 16001)] == \
        [0, 0, 1, 1, 2, 3, 98, 98]


def test_hann_window_values_and_sum():
    w = oa.hann_window()
    assert w.shape == (400,) and w[0] == 0.0 and abs(w[200] - 1.0) < 1e-15
    assert abs(w[100] - 0.5) < 1e-15 and abs(w[300] - 0.5) < 1e-15
    assert np.allclose(w[1:], w[1:][::-1], atol=1e-15)          # w[n] = w[400 - n]
    assert abs(w.sum() - 200.0) < 1e-12                          # a periodic Hann sums to N/2


def direct_dft_power(frame512: np.ndarray) -> np.ndarray:
    n = np.arange(512)
    out = np.empty(257)
    for k in range(257):
        ang = 2.0 * np.pi * k * n / 512.0
        re, im = np.sum(frame512 * np.cos(ang)), -np.sum(frame512 * np.sin(ang))
        out[k] = re * re + im * im
    return out


def test_power_spectrum_against_a_direct_dft_and_parseval():
    rng = np.random.default_rng(1)
    x = rng.uniform(-1, 1, size=400 + 2 * 160 + 7)              # three frames, ragged tail
    p = oa.power_spectrum(x)
    assert p.shape == (3, 257)
    w = 0.5 - 0.5 * np.cos(2 * np.pi * np.arange(400) / 400)
    for t in range(3):
        frame = np.zeros(512)
        frame[:400] = x[160 * t:160 * t + 400] * w
        assert np.allclose(p[t], direct_dft_power(frame), rtol=1e-10, atol=1e-12)
        # Parseval on the one-sided spectrum
        total = p[t, 0] + p[t, 256] + 2.0 * p[t, 1:256].sum()
        assert abs(total - 512.0 * np.sum(frame ** 2)) < 1e-8


def test_constant_signal_and_impulse():
    p = oa.power_spectrum(np.full(400, 0.25))
    assert abs(p[0, 0] - (0.25 * 200.0) ** 2) < 1e-9            # X[0] = c * sum(w)
    # an impulse at sample s lands at position s - 160 t of frame t: flat spectrum w[.]^2
    x = np.zeros(400 + 160 * 3)
    x[450] = 1.0
    p = oa.power_spectrum(x)
    w = oa.hann_window()
    for t, pos in ((0, None), (1, 290), (2, 130), (3, None)):
        want = 0.0 if pos is None else w[pos] ** 2
        assert np.allclose(p[t], want, atol=1e-12)


def test_mel_scale_and_corner_frequencies():
    assert abs(oa.hz_to_mel(1000.0) - 2595.0 * np.log10(1.0 + 1000.0 / 700.0)) < 1e-12
    assert abs(oa.hz_to_mel(1000.0) - 999.9855) < 1e-3
    assert abs(oa.mel_to_hz(oa.hz_to_mel(4321.0)) - 4321.0) < 1e-9
    assert oa.hz_to_mel(0.0) == 0.0


def test_mel_filters_are_unit_triangles_on_equal_mel_steps():
    fb = oa.mel_filterbank()
    assert fb.shape == (80, 257) and fb.min() >= 0.0 and fb.max() <= 1.0
    top = 2595.0 * np.log10(1.0 + 8000.0 / 700.0)
    corners = 700.0 * (10.0 ** (np.arange(82) * top / 81.0 / 2595.0) - 1.0)
    freqs = np.arange(257) * 16000.0 / 512.0
    for j in (0, 1, 17, 40, 79):
        want = np.interp(freqs, corners[j:j + 3], [0.0, 1.0, 0.0], left=0.0, right=0.0)
        assert np.allclose(fb[j], want, atol=1e-12)
    # neighbouring triangles sum to one between the first and the last centre
    inside = (freqs >= corners[1]) & (freqs <= corners[80])
    assert np.allclose(fb[:, inside].sum(axis=0), 1.0, atol=1e-12)
    assert np.all(fb[:, 0] == 0.0)                               # 0 Hz is the first filter's foot
    # a filter is zero outside its own corners
    assert np.all(fb[40][(freqs <= corners[40]) | (freqs >= corners[42])] == 0.0)


def test_log_mel_is_log_of_filtered_direct_spectrum():
    rng = np.random.default_rng(2)
    x = rng.normal(0, 0.1, size=560)
    w = 0.5 - 0.5 * np.cos(2 * np.pi * np.arange(400) / 400)
    fb = oa.mel_filterbank()                                      # pinned above
    got = oa.log_mel(x)
    assert got.shape == (80, 2)
    for t in range(2):
        frame = np.zeros(512)
        frame[:400] = x[160 * t:160 * t + 400] * w
        want = np.log(fb @ direct_dft_power(frame) + 2.0 ** -24)
        assert np.allclose(got[:, t], want, rtol=1e-10, atol=1e-10)
    # silence: every energy is the guard
    assert np.allclose(oa.log_mel(np.zeros(400)), np.log(2.0 ** -24))


def test_three_pass_normalisation():
    f = np.array([[1.0, 2.0, 3.0], [5.0, 5.0, 5.0], [-4.0, 0.0, 10.0]])
    got = oa.normalize(f)
    s0 = np.sqrt(2.0 / 3.0)
    assert np.allclose(got[0], np.array([-1.0, 0.0, 1.0]) / (s0 + 1e-5), atol=1e-14)
    assert np.all(got[1] == 0.0)                                 # constant feature
    m2 = 2.0
    v2 = ((-4 - m2) ** 2 + (0 - m2) ** 2 + (10 - m2) ** 2) / 3.0
    assert np.allclose(got[2], (f[2] - m2) / (np.sqrt(v2) + 1e-5), atol=1e-14)
    rng = np.random.default_rng(3)
    g = rng.normal(3.0, 2.0, size=(80, 57))
    n = oa.normalize(g)
    assert np.allclose(n.mean(axis=1), 0.0, atol=1e-12)
    sd = g.std(axis=1)
    assert np.allclose(n.std(axis=1), sd / (sd + 1e-5), atol=1e-12)
    assert np.allclose(oa.normalize(2.5 * g + 7.0), n, atol=1e-5)  # shift and scale drop out


def test_batch_layout_padding_and_independence():
    rng = np.random.default_rng(4)
    utts = [rng.normal(0, 0.1, size=n).astype(np.float32) for n in (2000, 399, 4000, 400)]
    out = oa.preprocess(utts)
    assert out.shape == (4, 80, oa.num_frames(4000))
    assert np.all(out[0, :, oa.num_frames(2000):] == 0.0)
    assert np.all(out[1] == 0.0)                                  # too short for one frame
    assert np.all(out[3, :, 1:] == 0.0) and np.all(out[3, :, 0] == 0.0)  # one frame: x - mean = 0
    for i in (0, 2):
        alone = oa.preprocess([utts[i]])[0]
        assert np.array_equal(out[i, :, :alone.shape[1]], alone)
    raw = oa.preprocess(utts, normalized=False)
    assert np.array_equal(raw[2], oa.log_mel(utts[2]))
