"""Synthetic uint8 image batches with natural-image-like smoothness.

Recipe per image: three independent N(0,1) noise fields (R, G, B) are blurred with a separable
Gaussian (standard deviation `sigma` pixels, truncated at +-3 sigma, periodic wrap), the image is
rescaled to empirical mean 120 and standard deviation 60, N(0, 8^2) pixel noise is added, and the
result is rounded half up and clamped to 0..255.
"""
import numpy as np

from .rng import Stream


def _gauss_kernel(sigma):
    r = int(np.ceil(3.0 * sigma))
    t = np.arange(-r, r + 1, dtype=np.float64)
    k = np.exp(-0.5 * (t / sigma) ** 2)
    return k / k.sum(), r


def _blur_wrap(f, sigma):
    """Separable periodic Gaussian blur over the last two axes."""
    k, r = _gauss_kernel(sigma)
    out = np.zeros_like(f)
    for d, w in zip(range(-r, r + 1), k):
        out += w * np.roll(f, d, axis=-1)
    f2 = np.zeros_like(f)
    for d, w in zip(range(-r, r + 1), k):
        f2 += w * np.roll(out, d, axis=-2)
    return f2


def smooth_field_images(seed, batch, height, width, sigma, channels=3):
    """uint8 [batch, channels, height, width] (NCHW)."""
    n = batch * channels * height * width
    base = Stream(seed, "image/field").normal(n).reshape(batch, channels, height, width)
    noise = Stream(seed, "image/noise").normal(n).reshape(batch, channels, height, width)
    f = _blur_wrap(base, float(sigma))
    mean = f.mean(axis=(1, 2, 3), keepdims=True)
    std = f.std(axis=(1, 2, 3), keepdims=True)
    f = (f - mean) / np.maximum(std, 1e-12) * 60.0 + 120.0 + 8.0 * noise
    return np.clip(np.floor(f + 0.5), 0, 255).astype(np.uint8)
