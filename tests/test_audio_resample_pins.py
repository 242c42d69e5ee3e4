"""Pins for the Resample oracle: what the mathematics fixes about a Hann-windowed sinc
interpolator (zero crossings, peak, support, symmetry), exact covariances, the polyphase
structure against scipy's upfirdn, and pass-band / stop-band behaviour."""
from __future__ import annotations

from math import gcd

import numpy as np
import pytest

from oracle import audio as oa


@pytest.mark.parametrize("rin,rout", [(48000, 16000), (44100, 16000), (8000, 16000), (16000, 16000)])
def test_kernel_zero_crossings_peak_support_symmetry(rin, rout):
    fc = 0.99 * min(1.0, rout / rin)
    assert abs(oa.resample_kernel(0.0, rin, rout) - fc) < 1e-15          # h(0) = fc
    k = np.arange(1, 6)
    assert np.max(np.abs(oa.resample_kernel(k / fc, rin, rout))) < 1e-15   # sinc zeros at k / fc
    assert oa.resample_kernel(6.0 / fc, rin, rout) == 0.0                # support |fc t| < 6
    assert oa.resample_kernel(6.0 / fc + 0.3, rin, rout) == 0.0
    t = np.linspace(0.01, 6.0 / fc, 97)
    assert np.allclose(oa.resample_kernel(t, rin, rout), oa.resample_kernel(-t, rin, rout), atol=1e-16)
    # half-way to the first zero: fc * sinc(1/2) * cos^2(pi/24) = fc * (2/pi) * cos^2(pi/24)
    want = fc * (2.0 / np.pi) * np.cos(np.pi / 24.0) ** 2
    assert abs(oa.resample_kernel(0.5 / fc, rin, rout) - want) < 1e-14
    # the integral of h is (nearly) one: unit gain at 0 Hz
    tt = np.linspace(-6.0 / fc, 6.0 / fc, 200001)
    assert abs(np.trapezoid(oa.resample_kernel(tt, rin, rout), tt) - 1.0) < 2e-3


def test_output_length_and_linearity():
    assert oa.resampled_length(48000, 48000, 16000) == 16000
    assert oa.resampled_length(44101, 44100, 16000) == 16001             # ceil
    assert oa.resampled_length(0, 44100, 16000) == 0
    rng = np.random.default_rng(1)
    a, b = rng.normal(size=700), rng.normal(size=700)
    ya, yb = oa.resample(a, 44100, 16000), oa.resample(b, 44100, 16000)
    assert np.allclose(oa.resample(2.0 * a - 3.0 * b, 44100, 16000), 2.0 * ya - 3.0 * yb, atol=1e-12)


@pytest.mark.parametrize("rin,rout", [(48000, 16000), (44100, 16000), (8000, 16000), (22050, 16000)])
def test_shift_by_one_period_of_the_ratio_is_exact(rin, rout):
    """Delaying the input by orig samples delays the output by new samples, exactly."""
    g = gcd(rin, rout)
    orig, new = rin // g, rout // g
    rng = np.random.default_rng(2)
    x = rng.normal(size=3 * orig + 400)
    y = oa.resample(x, rin, rout)
    yd = oa.resample(np.concatenate([np.zeros(orig), x]), rin, rout)
    assert np.allclose(yd[new:new + y.size], y, atol=1e-13)


@pytest.mark.parametrize("rin,rout", [(48000, 16000), (44100, 16000), (8000, 16000)])
def test_polyphase_structure_against_upfirdn(rin, rout):
    """The same filter sampled on the fine grid (spacing 1/new input samples), run through
    scipy.signal.upfirdn(up=new, down=orig): a library routine for exactly this sum."""
    from scipy.signal import upfirdn

    g = gcd(rin, rout)
    orig, new = rin // g, rout // g
    fc = 0.99 * min(1.0, new / orig)
    reach = int(np.ceil(6.0 / fc)) + 1
    fine = np.arange(-reach * new, reach * new + 1)                      # in units of 1/new samples
    taps = oa.resample_kernel(fine / new, rin, rout)
    rng = np.random.default_rng(3)
    x = rng.normal(size=2 * orig + 300)
    full = upfirdn(taps, x, up=new, down=1)                              # fine-grid convolution
    want = full[reach * new::orig][:oa.resampled_length(x.size, rin, rout)]
    got = oa.resample(x, rin, rout)
    assert np.allclose(got, want[:got.size], atol=1e-12)


def tone(freq, rate, n):
    return np.sin(2 * np.pi * freq * np.arange(n) / rate + 0.3)


def test_pass_band_tones_survive_and_out_of_band_tones_vanish():
    """48 kHz -> 16 kHz: cutoff 7.92 kHz; the Hann window of twelve zero crossings puts a
    transition band of about +-1.3 kHz around it and keeps side lobes below -44 dB beyond."""
    n_in = 48000 // 4
    inner = slice(60, -60)                                               # away from the zero-padded ends
    for f, bound in ((100.0, 1e-3), (1000.0, 1e-3), (3000.0, 1e-3), (5000.0, 1e-2)):
        y = oa.resample(tone(f, 48000, n_in), 48000, 16000)
        want = tone(f, 16000, y.size)
        assert np.max(np.abs(y[inner] - want[inner])) < bound
    for f, bound in ((11000.0, 6.3e-3), (15000.0, 6.3e-3), (20000.0, 6.3e-3)):  # -44 dB
        y = oa.resample(tone(f, 48000, n_in), 48000, 16000)
        assert np.max(np.abs(y[inner])) < bound
    # upsampling keeps a tone below the old Nyquist
    y = oa.resample(tone(1000.0, 8000, 2000), 8000, 16000)              # a quarter of the cutoff
    want = tone(1000.0, 16000, y.size)
    assert np.max(np.abs(y[inner] - want[inner])) < 1e-3


def test_impulse_lands_where_the_position_arithmetic_says():
    """x = delta[n0]: the largest output is the one whose position m * rin / rout is nearest
    n0, and equal rates with an integer position reproduce fc at the sample itself."""
    x = np.zeros(300)
    x[120] = 1.0
    y = oa.resample(x, 48000, 16000)
    assert int(np.argmax(y)) == 40 and abs(y[40] - 0.99 / 3.0) < 1e-12  # position 40 * 3 = 120
    y = oa.resample(x, 8000, 16000)
    assert int(np.argmax(y)) == 240 and abs(y[240] - 0.99) < 1e-12      # position 240 / 2 = 120
    y = oa.resample(x, 44100, 16000)
    assert int(np.argmax(y)) == round(120 * 16000 / 44100)
