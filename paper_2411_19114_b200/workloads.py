"""Seeded synthetic image workloads (inputs only — none of the transform's arithmetic).

These stand in for the decoded ImageNet-style images the paper's vision
servers receive (Sec. 5, "Input query modeling"): same shapes, sizes and value
distributions, no dataset item.  Both the tests' CPU checker and the CUDA path
read their inputs from here, so the two see identical bytes.

Image sizes are written W x H in the workload descriptions (320x240 is 240 rows
of 320 pixels); arrays are HWC uint8.
"""
from __future__ import annotations

from concurrent.futures import ThreadPoolExecutor

import numpy as np

MEAN = (0.485, 0.456, 0.406)
STD = (0.229, 0.224, 0.225)
RESIZE_SHORT = 256
OUT_SIZE = 224


def uniform_image(rng: np.random.Generator, h: int, w: int) -> np.ndarray:
    """Bytes i.i.d. uniform on 0..255."""
    return rng.integers(0, 256, size=(h, w, 3), dtype=np.uint8)


def _blur_axis(a: np.ndarray, axis: int, kernel: np.ndarray) -> np.ndarray:
    r = len(kernel) // 2
    pad = [(0, 0)] * a.ndim
    pad[axis] = (r, r)
    p = np.pad(a, pad, mode="edge")
    out = np.zeros_like(a)
    n = a.shape[axis]
    for t, kv in enumerate(kernel):
        sl = [slice(None)] * a.ndim
        sl[axis] = slice(t, t + n)
        out += kv * p[tuple(sl)]
    return out


def smooth_image(rng: np.random.Generator, h: int, w: int, sigma: float = 3.0,
                 jitter: float = 8.0) -> np.ndarray:
    """Smooth value noise: a uniform[0,255] field per channel, separable Gaussian
    blur (sigma 3 px, radius 9, edge clamp) in float64, plus uniform jitter in
    [-8, 8], rounded and clipped to 0..255.  No contrast stretch."""
    field = rng.uniform(0.0, 255.0, size=(h, w, 3))
    r = int(3 * sigma)
    t = np.arange(-r, r + 1, dtype=np.float64)
    kernel = np.exp(-0.5 * (t / sigma) ** 2)
    kernel /= kernel.sum()
    field = _blur_axis(_blur_axis(field, 0, kernel), 1, kernel)
    field += rng.uniform(-jitter, jitter, size=(h, w, 3))
    return np.clip(np.rint(field), 0, 255).astype(np.uint8)


def _per_image(seed: int, sizes, kind: str, workers: int = 8) -> list[np.ndarray]:
    """One child generator per image (spawned from the seed), so that any prefix
    of the list is the same whatever its length."""
    children = np.random.SeedSequence(seed).spawn(len(sizes))
    make = uniform_image if kind == "uniform" else smooth_image

    def one(i):
        h, w = sizes[i]
        return make(np.random.default_rng(children[i]), h, w)

    if len(sizes) <= 2 or workers <= 1:
        return [one(i) for i in range(len(sizes))]
    with ThreadPoolExecutor(max_workers=workers) as ex:
        return list(ex.map(one, range(len(sizes))))


def fixed_size_batch(seed: int, n: int, h: int, w: int, kind: str) -> list[np.ndarray]:
    return _per_image(seed, [(h, w)] * n, kind)


def mixed_sizes(seed: int, n: int, lo: int = 240, hi: int = 500) -> list[tuple[int, int]]:
    """H and W independent uniform integers in [lo, hi] per image."""
    rng = np.random.default_rng(seed)
    hw = rng.integers(lo, hi + 1, size=(n, 2))
    return [(int(a), int(b)) for a, b in hw]


def uniform_320x240(n: int = 64, seed: int = 1) -> list[np.ndarray]:
    """n images of 320x240 with uniform random bytes (fp32 output case)."""
    return fixed_size_batch(seed, n, 240, 320, "uniform")


def mixed_smooth(n: int = 256, seed: int = 2) -> list[np.ndarray]:
    """n images, H and W uniform in [240, 500], smooth noise: the ragged batch."""
    return _per_image(seed, mixed_sizes(seed, n), "smooth")


def server_batch_500x375(stream: int, n: int = 32) -> list[np.ndarray]:
    """One small server's batch of 500x375 smooth-noise images (seed 30 + stream)."""
    return fixed_size_batch(30 + stream, n, 375, 500, "smooth")


def hires_1080p(n: int = 64, seed: int = 4) -> list[np.ndarray]:
    """n images of 1920x1080, smooth noise plus jitter (heavy downscale case)."""
    return fixed_size_batch(seed, n, 1080, 1920, "smooth")


def sweep_500x375(n: int = 2048, seed: int = 5) -> list[np.ndarray]:
    """n images of 500x375 with uniform random bytes; prefixes serve the batch sweep."""
    return fixed_size_batch(seed, n, 375, 500, "uniform")


# ---- audio: seeded synthetic utterances (inputs only) -------------------------------------------

AUDIO_RATE = 16000


def utterance(rng: np.random.Generator, seconds: float) -> np.ndarray:
    """A speech-like test signal: a handful of harmonics of a slowly gliding pitch under a
    syllable-rate envelope, plus white noise 40 dB below; float32 in [-1, 1] at 16 kHz.
    It stands in for the read speech of the paper's audio corpus (Sec. 5): broadband, with
    pauses; no corpus item is reproduced."""
    n = int(round(seconds * AUDIO_RATE))
    t = np.arange(n, dtype=np.float64) / AUDIO_RATE
    f0 = rng.uniform(90.0, 220.0)
    glide = 1.0 + 0.15 * np.sin(2 * np.pi * rng.uniform(0.2, 0.7) * t + rng.uniform(0, 6.28))
    phase = 2 * np.pi * np.cumsum(f0 * glide) / AUDIO_RATE
    x = np.zeros(n)
    for h in range(1, 24):
        x += rng.uniform(0.2, 1.0) / h * np.sin(h * phase + rng.uniform(0, 6.28))
    env = np.clip(np.sin(2 * np.pi * rng.uniform(2.0, 4.0) * t + rng.uniform(0, 6.28)), 0.0, 1.0)
    x = x * env ** 2
    x = 0.5 * x / max(1e-9, np.max(np.abs(x)))
    x += 0.005 * rng.standard_normal(n)
    return np.clip(x, -1.0, 1.0).astype(np.float32)


def utterances(n: int, seed: int, min_s: float = 1.5, max_s: float = 15.0) -> list[np.ndarray]:
    """n utterances with lengths uniform in [min_s, max_s] seconds (a ragged batch)."""
    seqs = np.random.SeedSequence(seed).spawn(n + 1)
    lens = np.random.default_rng(seqs[0]).uniform(min_s, max_s, size=n)
    return [utterance(np.random.default_rng(seqs[i + 1]), float(lens[i])) for i in range(n)]


def jpeg_streams(images, quality: int = 90, subsampling: int = 2, restart_rows: int = 1):
    """The images as baseline JPEG streams written by an image library (the input of the Decode
    unit): chroma subsampling 0 (4:4:4), 1 (4:2:2) or 2 (4:2:0), a restart marker every
    ``restart_rows`` rows of MCUs (0: none).  Stand-ins for the compressed files of the paper's
    image workload; the content is the seeded synthetic images given."""
    import io

    from PIL import Image

    out = []
    for im in images:
        buf = io.BytesIO()
        extra = {"restart_marker_rows": restart_rows} if restart_rows else {}
        Image.fromarray(im).save(buf, format="JPEG", quality=quality, subsampling=subsampling, **extra)
        out.append(buf.getvalue())
    return out
