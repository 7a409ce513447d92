"""Seeded synthetic inputs shaped like the paper's Llama-family layers.

Holds no arithmetic of the method: only random draws (numpy ``Generator(PCG64(seed))``) and the
storage cast to bfloat16 (round to nearest even), so that the CUDA path and the CPU oracle
can be fed the identical bits.  bfloat16 tensors are returned as ``uint16`` bit patterns.
"""
from __future__ import annotations

import numpy as np


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round binary32 to bfloat16 (nearest even); returns the uint16 bit patterns."""
    w = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    # w + 0x7FFF + (bit 16 of w), in 32-bit arithmetic: the sum fits for every finite value and infinity
    # (at most 0xFF800000 + 0x8000); only NaN patterns at the very top of the range need the wide path
    if w.size and int(w.max()) >= 0xFFFF0000:
        w64 = w.astype(np.uint64)
        return ((w64 + 0x7FFF + ((w64 >> 16) & 1)) >> 16).astype(np.uint16)
    inc = (w >> np.uint32(16)) & np.uint32(1)
    inc += np.uint32(0x7FFF)
    inc += w
    inc >>= np.uint32(16)
    return inc.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


def _rng(seed: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(seed))


def gaussian_with_outliers(rows: int, cols: int, rng, frac: float = 0.01, gain: float = 20.0):
    """N(0,1) with a Bernoulli(frac) subset of entries multiplied by ``gain`` (binary32)."""
    a = rng.standard_normal((rows, cols), dtype=np.float32)
    hit = rng.random((rows, cols)) < frac
    return np.where(hit, a * np.float32(gain), a).astype(np.float32)


def channel_scaled_gaussian(rows: int, cols: int, rng, lo: float = 0.5, hi: float = 8.0):
    """N(0,1) times a per-channel scale drawn log-uniform in [lo, hi] (outlier channels)."""
    c = np.exp(rng.uniform(np.log(lo), np.log(hi), size=cols)).astype(np.float32)
    return rng.standard_normal((rows, cols), dtype=np.float32) * c[None, :]


def student_t(rows: int, cols: int, rng, nu: float = 4.0):
    return rng.standard_t(nu, size=(rows, cols)).astype(np.float32)


def weights(rows: int, cols: int, rng, std: float = 0.02):
    return (rng.standard_normal((rows, cols), dtype=np.float32) * np.float32(std)).astype(np.float32)


def config1(seed: int = 0):
    """Single W4A4 linear, binary32: X[256x512], W[512x512], N(0,1) with 1% x20 outliers."""
    rng = _rng(seed)
    x = gaussian_with_outliers(256, 512, rng)
    w = gaussian_with_outliers(512, 512, rng)
    return {"x": x, "w": w, "bits": 4, "had_block": 512, "trust_factor": 1.0, "dtype": "f32"}


def config2(seed: int = 1, tokens: int = 4096, hidden: int = 2048, out: int = 2048):
    """1.6B-scale layer, bfloat16: channel-scaled Gaussian activations, N(0, 0.02^2) weights."""
    rng = _rng(seed)
    x = f32_to_bf16_bits(channel_scaled_gaussian(tokens, hidden, rng))
    w = f32_to_bf16_bits(weights(out, hidden, rng))
    return {"x": x, "w": w, "dtype": "bf16"}


def config4(seed: int = 2, tokens: int = 8192, hidden: int = 2048, inter: int = 5504):
    """Llama-style MLP block at 1.6B scale, bfloat16: Student-t(4) activations."""
    rng = _rng(seed)
    return {
        "x": f32_to_bf16_bits(student_t(tokens, hidden, rng)),
        "w_gate": f32_to_bf16_bits(weights(inter, hidden, rng)),
        "w_up": f32_to_bf16_bits(weights(inter, hidden, rng)),
        "w_down": f32_to_bf16_bits(weights(hidden, inter, rng)),
        "dtype": "bf16",
    }


def config5_point(index: int, tokens: int, hidden: int, seed: int = 3):
    """One point of the bit-width / shape sweep: Student-t(4) activations, square weights."""
    rng = _rng(seed + index)
    return {"x": f32_to_bf16_bits(student_t(tokens, hidden, rng)),
            "w": f32_to_bf16_bits(weights(hidden, hidden, rng)), "dtype": "bf16"}
