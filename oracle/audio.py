"""TEST INFRASTRUCTURE ONLY: CPU oracle of the audio preprocessing path (numpy, float64).

The paper lists the audio units as Resample, Mel spectrogram and Normalize (Table 1) and the
operations as resampling, a Fourier transform and a Mel filterbank (Sec. 2.3 item 1); Sec. 4.2 spells out Normalize as three passes: the mean over all samples, the
variance using that mean, then the normalisation of each sample by both.  It fixes no numerics.
The readings taken here (every one of them a choice of this library, not of the paper):

  - input: mono float32 PCM at the model's rate (16 kHz); other rates go through `resample` below;
  - framing: frame t holds samples [t*hop, t*hop + win), win = 400, hop = 160, no padding, so an
    utterance of L >= win samples gives T = 1 + (L - win) // hop frames (none when L < win);
  - window: periodic Hann, w[n] = 0.5 - 0.5*cos(2*pi*n/win); the windowed frame is zero-padded to
    n_fft = 512;
  - spectrum: power |X[k]|^2 of the one-sided DFT, k = 0 .. n_fft/2;
  - Mel filters: n_mels = 80 triangles on the HTK mel scale m(f) = 2595*log10(1 + f/700) between
    0 Hz and rate/2, corner frequencies equally spaced in mel; filter j has weight
    max(0, min((f - f_j)/(f_{j+1} - f_j), (f_{j+2} - f)/(f_{j+2} - f_{j+1}))) at bin frequency
    f = k*rate/n_fft; no area normalisation;
  - log: natural logarithm of (mel energy + 2^-24);
  - Normalize: per utterance and per Mel filter, over that utterance's T frames:
    (x - mean)/(sqrt(var) + 1e-5) with var the mean squared deviation (divide by T);
  - output: [n, n_mels, T_max] float32, frames beyond an utterance's T are 0.

Only the DFT is a library routine (numpy.fft.rfft); everything else is written out.  The module
shares nothing with the CUDA path.  Every function is pinned by tests that do not use it to make
their expected values (tests/test_audio_oracle_pins.py): none is "parity unpinned".
"""
from __future__ import annotations

import numpy as np

RATE = 16000
WIN = 400
HOP = 160
N_FFT = 512
N_MELS = 80
LOG_GUARD = 2.0 ** -24
STD_GUARD = 1e-5


def num_frames(length: int) -> int:
    """Frames of an utterance of `length` samples (framing reading above)."""
    return 0 if length < WIN else 1 + (length - WIN) // HOP


def hann_window() -> np.ndarray:
    n = np.arange(WIN, dtype=np.float64)
    return 0.5 - 0.5 * np.cos(2.0 * np.pi * n / WIN)


def hz_to_mel(f):
    return 2595.0 * np.log10(1.0 + np.asarray(f, dtype=np.float64) / 700.0)


def mel_to_hz(m):
    return 700.0 * (10.0 ** (np.asarray(m, dtype=np.float64) / 2595.0) - 1.0)


def mel_filterbank() -> np.ndarray:
    """[N_MELS, N_FFT/2 + 1] triangle weights."""
    corners = mel_to_hz(np.linspace(hz_to_mel(0.0), hz_to_mel(RATE / 2.0), N_MELS + 2))
    freqs = np.arange(N_FFT // 2 + 1, dtype=np.float64) * RATE / N_FFT
    fb = np.zeros((N_MELS, N_FFT // 2 + 1), dtype=np.float64)
    for j in range(N_MELS):
        lo, mid, hi = corners[j], corners[j + 1], corners[j + 2]
        up = (freqs - lo) / (mid - lo)
        down = (hi - freqs) / (hi - mid)
        fb[j] = np.maximum(0.0, np.minimum(up, down))
    return fb


def power_spectrum(samples: np.ndarray) -> np.ndarray:
    """[T, N_FFT/2 + 1]: |DFT|^2 of every windowed, zero-padded frame of one utterance."""
    x = np.asarray(samples, dtype=np.float64)
    t = num_frames(x.size)
    w = hann_window()
    frames = np.zeros((t, N_FFT), dtype=np.float64)
    for i in range(t):
        frames[i, :WIN] = x[i * HOP:i * HOP + WIN] * w
    spec = np.fft.rfft(frames, n=N_FFT, axis=1)
    return spec.real ** 2 + spec.imag ** 2


def log_mel(samples: np.ndarray) -> np.ndarray:
    """[N_MELS, T]: log Mel energies of one utterance, before normalisation."""
    return np.log(power_spectrum(samples) @ mel_filterbank().T + LOG_GUARD).T


def normalize(feat: np.ndarray) -> np.ndarray:
    """Sec. 4.2's three passes, per Mel filter over the frames: mean, variance from that mean,
    then (x - mean)/(sqrt(var) + guard)."""
    if feat.shape[1] == 0:
        return feat.copy()
    mean = feat.sum(axis=1, keepdims=True) / feat.shape[1]
    var = ((feat - mean) ** 2).sum(axis=1, keepdims=True) / feat.shape[1]
    return (feat - mean) / (np.sqrt(var) + STD_GUARD)


def preprocess(utterances: list[np.ndarray], normalized: bool = True) -> np.ndarray:
    """[n, N_MELS, T_max] float64 for a ragged batch of utterances; frames past an utterance's
    own count are 0."""
    counts = [num_frames(len(u)) for u in utterances]
    t_max = max(counts) if counts else 0
    out = np.zeros((len(utterances), N_MELS, t_max), dtype=np.float64)
    for i, u in enumerate(utterances):
        if counts[i]:
            f = log_mel(u)
            out[i, :, :counts[i]] = normalize(f) if normalized else f
    return out


# ---- Resample (Table 1's first audio unit): bandlimited interpolation --------------------------------
#
# The paper only names the unit ("resampling", Sec. 2.3 item 1).  Reading: the classical
# bandlimited interpolation with a Hann-windowed sinc (J. O. Smith, "Digital Audio Resampling"),
# six zero crossings each side, cutoff at 0.99 of the lower of the two Nyquist frequencies:
#   y[m] = sum_n x[n] * h(n - m * rate_in / rate_out),      M = ceil(L * rate_out / rate_in) outputs,
#   h(t) = fc * sinc(fc * t) * cos^2(pi * fc * t / (2 * Z))  for |fc * t| < Z, else 0,
#   fc = 0.99 * min(1, rate_out / rate_in),  Z = 6,  sinc(u) = sin(pi u) / (pi u),
# samples outside the utterance count as 0.  It is an approximation of ideal bandlimited
# interpolation; the pins check what the mathematics fixes about it (zero crossings, peak,
# support and symmetry of h, exact shift covariance, the polyphase structure against a library
# routine, pass-band and stop-band behaviour within the window's known bounds).

RESAMPLE_ZEROS = 6
RESAMPLE_ROLLOFF = 0.99


def resample_kernel(t, rate_in: int, rate_out: int):
    """h(t) for t in input-sample units (float64 array)."""
    t = np.asarray(t, dtype=np.float64)
    fc = RESAMPLE_ROLLOFF * min(1.0, rate_out / rate_in)
    u = fc * t
    inside = np.abs(u) < RESAMPLE_ZEROS
    window = np.cos(np.pi * u / (2.0 * RESAMPLE_ZEROS)) ** 2
    return np.where(inside, fc * np.sinc(u) * window, 0.0)


def resampled_length(length: int, rate_in: int, rate_out: int) -> int:
    return -(-length * rate_out // rate_in)


def resample(samples: np.ndarray, rate_in: int, rate_out: int) -> np.ndarray:
    """The resampled utterance (float64), straight from the definition."""
    from math import gcd

    x = np.asarray(samples, dtype=np.float64)
    g = gcd(rate_in, rate_out)
    orig, new = rate_in // g, rate_out // g
    m_count = resampled_length(x.size, rate_in, rate_out)
    fc = RESAMPLE_ROLLOFF * min(1.0, new / orig)
    reach = int(np.ceil(RESAMPLE_ZEROS / fc)) + 1
    out = np.zeros(m_count, dtype=np.float64)
    for m in range(m_count):
        centre = m * orig // new                      # floor of the position in input samples
        frac = (m * orig % new) / new                 # exact position = centre + frac
        n = np.arange(centre - reach, centre + reach + 2)
        ok = (n >= 0) & (n < x.size)
        h = resample_kernel((n - centre) - frac, rate_in, rate_out)
        out[m] = np.sum(x[n[ok]] * h[ok])
    return out
