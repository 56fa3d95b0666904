"""Independent numpy routines the oracle is pinned against (no oracle code here)."""
from __future__ import annotations

import numpy as np

from paper_2604_16429_b200 import synth


def f64(bits: np.ndarray) -> np.ndarray:
    return synth.bf16_bits_to_f32(bits).astype(np.float64)


def quantised(shape, rng, step=1 / 16, lim=2.0) -> np.ndarray:
    """bf16 bits of values that are multiples of `step` in [-lim, lim): exactly
    representable, and still representable after adding +-step/2 or +-step/4."""
    n = int(round(lim / step))
    vals = rng.integers(-n, n, size=shape).astype(np.float32) * np.float32(step)
    bits = synth.to_bf16_bits(vals)
    assert np.array_equal(synth.bf16_bits_to_f32(bits), vals)
    return bits


def dense_attention(q, k, v, scale):
    """Textbook softmax attention of every query over every key, fp64."""
    x = scale * (q @ k.T)
    x = x - x.max(axis=1, keepdims=True)
    p = np.exp(x)
    z = p.sum(axis=1, keepdims=True)
    return (p / z) @ v, np.log(z[:, 0]) + (scale * (q @ k.T)).max(axis=1)


def block_tokens(nlon, bh, bw, nbw, j):
    by, bx = divmod(j, nbw)
    r = np.arange(bh)[:, None] + by * bh
    c = np.arange(bw)[None, :] + bx * bw
    return (r * nlon + c).reshape(-1)


def local_blocks(by, bx, nbh, nbw, rlat=1, rlon=1):
    """Local neighbourhood as a python set, written straight from its definition."""
    return {min(max(by + dy, 0), nbh - 1) * nbw + (bx + dx) % nbw
            for dy in range(-rlat, rlat + 1) for dx in range(-rlon, rlon + 1)}
