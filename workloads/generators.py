"""Seeded synthetic tensors shaped like the paper's workloads.

This module serves both the CPU oracle and the CUDA path and therefore holds none of
the method's arithmetic: it only draws random numbers.  Raw images are uint8, float
weights are float32 draws from N(0, 0.05) (the paper observes that convolution kernels
are roughly zero-mean normal, Section 3.1), biases are int32 in [-2^12, 2^12].

Every image is generated from its own (seed, index) stream so that a single image of a
large batch can be produced alone.
"""
import numpy as np


def _box_blur_axis(a, radius, axis):
    k = 2 * radius + 1
    pad = [(0, 0)] * a.ndim
    pad[axis] = (radius + 1, radius)
    c = np.cumsum(np.pad(a, pad, mode="edge"), axis=axis)
    n = a.shape[axis]
    hi = np.take(c, np.arange(k, k + n), axis=axis)
    lo = np.take(c, np.arange(0, n), axis=axis)
    return (hi - lo) / k


def smooth_image(seed: int, index: int, h: int, w: int, c: int) -> np.ndarray:
    """One uint8 image [h][w][c]: low-passed Gaussian noise (std 40 around 128) plus eight
    axis-aligned rectangles of +-40 (edges), clipped to [0, 255]."""
    rng = np.random.default_rng([int(seed), 1000, int(index)])
    img = rng.standard_normal((h, w, c))
    for _ in range(3):
        img = _box_blur_axis(img, 4, 0)
        img = _box_blur_axis(img, 4, 1)
    std = img.std(axis=(0, 1), keepdims=True)
    img = img / np.maximum(std, 1e-12) * 40.0 + 128.0
    for _ in range(8):
        y0, y1 = np.sort(rng.integers(0, h + 1, size=2))
        x0, x1 = np.sort(rng.integers(0, w + 1, size=2))
        amp = 40.0 if rng.integers(0, 2) else -40.0
        img[y0:y1, x0:x1, :] += amp
    return np.clip(np.floor(img + 0.5), 0, 255).astype(np.uint8)


def image_batch(seed: int, n: int, h: int, w: int, c: int, first: int = 0) -> np.ndarray:
    """uint8 [n][h][w][c]; image i is ``smooth_image(seed, first + i, ...)``."""
    out = np.empty((n, h, w, c), dtype=np.uint8)
    for i in range(n):
        out[i] = smooth_image(seed, first + i, h, w, c)
    return out


def uniform_u8(seed: int, shape) -> np.ndarray:
    rng = np.random.default_rng([int(seed), 2000])
    return rng.integers(0, 256, size=shape, dtype=np.uint8)


def weights_f(seed: int, layer: int, c_out: int, kh: int, kw: int, c_in: int) -> np.ndarray:
    """float32 [c_out][kh][kw][c_in] ~ N(0, 0.05)."""
    rng = np.random.default_rng([int(seed), 3000, int(layer)])
    return rng.normal(0.0, 0.05, size=(c_out, kh, kw, c_in)).astype(np.float32)


def bias_i32(seed: int, layer: int, c_out: int) -> np.ndarray:
    """int32 [c_out] uniform in [-4096, 4096]."""
    rng = np.random.default_rng([int(seed), 4000, int(layer)])
    return rng.integers(-4096, 4097, size=(c_out,), dtype=np.int32)
