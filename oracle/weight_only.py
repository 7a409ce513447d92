"""Weight-only QuEST forward (Section 4.5, "Weight-only quantization"), written out step by step.

TEST INFRASTRUCTURE ONLY.  The paper trains models whose weights are quantized to 1-4 bits while
the activations keep 16 bits, and gives no separate algorithm for it.

READING: Algorithm 1 with the rounding of the activations left out.  The weights take their two
steps unchanged (rotation, then RMS scale and rounding to the b-bit grid: ``quest_oracle.quantize``).
The activations are rotated by the same orthonormal block Hadamard transform and stored as
bfloat16, the 16-bit activation type of the paper's runs:

    x_h[m, :] = bf16( fl32( u[m, :] * fl32(1 / sqrt(g)) ) ),   u = binary32 butterflies of x in the
                                                               quantizer's order (``fwht_block``)
    y[m, n]   = sw[n] * sum_k x_h[m, k] * c_w[n, k],           c_w = 2 k_w - (2^b - 1)

Because the transform is orthonormal, this equals x times the dequantised weights taken back to the
original basis, y = x (IHT(w_q_h))^T, up to the bfloat16 rounding of x_h; the tests pin that
identity.  The products are evaluated exactly in binary64 here; the CUDA path accumulates in
binary32 and is held to a bound derived from that (tests/test_gpu_weight_only.py).
Pins: tests/test_oracle_weight_only.py.
"""
from __future__ import annotations

import numpy as np

from . import quest_oracle as qo


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.asarray(b, np.uint16).astype(np.uint32) << 16).view(np.float32)


def f32_to_bf16_bits(v: np.ndarray) -> np.ndarray:
    """Round binary32 to bfloat16, ties to even (finite inputs)."""
    u = np.ascontiguousarray(v, dtype=np.float32).view(np.uint32).astype(np.uint64)
    lsb = (u >> 16) & 1
    return ((u + 0x7FFF + lsb) >> 16).astype(np.uint16)


def rotate_bf16(x: np.ndarray, g: int) -> np.ndarray:
    """x [M, K] (float32, or uint16 holding bfloat16 bits) -> bfloat16 bits of HT(x), blocks of g."""
    xf = bf16_bits_to_f32(x) if x.dtype == np.uint16 else np.asarray(x, np.float32)
    M, K = xf.shape
    assert K % g == 0
    inv = np.float32(1.0) / np.sqrt(np.float32(g))
    out = np.empty((M, K), np.uint16)
    for m in range(M):
        for j in range(0, K, g):
            u = qo.fwht_block(xf[m, j:j + g])                       # binary32, canonical butterfly order
            out[m, j:j + g] = f32_to_bf16_bits(u * inv)              # one binary32 product, then one rounding
    return out


def linear_fwd_weight_only(x: np.ndarray, w: np.ndarray, bits_w: int, had_block: int,
                           trust_factor: float = 1.0) -> dict:
    """Returns xh (bfloat16 bits), wq / sw / mw of the weight quantizer, y (float64), and
    ``bound`` = sw[n] * sum_k |x_h c_w| per output (the magnitude a binary32 accumulation error scales with)."""
    q = qo.quantize(w, bits_w, had_block, trust_factor)
    K = x.shape[1]
    cw = qo.unpack_grid_values(q["codes"], K, bits_w).astype(np.float64)
    xh_bits = rotate_bf16(x, had_block)
    xh = bf16_bits_to_f32(xh_bits).astype(np.float64)
    sw = q["scales"].astype(np.float64)
    y = (xh @ cw.T) * sw[None, :]
    bound = (np.abs(xh) @ np.abs(cw).T) * sw[None, :]
    return {"xh": xh_bits, "wq": q["codes"], "sw": q["scales"], "mw": q["mask"], "y": y, "bound": bound}
