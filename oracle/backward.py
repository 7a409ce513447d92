"""QuEST training backward (Algorithm 2) written out from its definition, in binary64 numpy.

TEST INFRASTRUCTURE ONLY.  Inputs are what the forward pass returns (packed codes, per-row scales,
trust-mask bitmaps) and the gradient dL/dy:

    dL/dxq_h = dL/dy  wq_h                       (activation-gradient product)
    dL/dx    = IHT( M(x_h; xq_h) * dL/dxq_h )    (trust mask, inverse transform)
    dL/dwq_h = dL/dy^T xq_h                      (weight-gradient product)
    dL/dw    = IHT( M(w_h; wq_h) * dL/dwq_h )    (trust mask, inverse transform)

with xq_h = sx[m] * c_x[m, k] and wq_h = sw[n] * c_w[n, k] the dequantised grid values in the
orthonormal Hadamard domain (c = 2k - (2^b - 1)), and IHT the inverse of the orthonormal
block-diagonal Hadamard transform of Eq. 2: the Sylvester matrix is symmetric, so IHT = HT =
H_g / sqrt(g) on every block of g elements.

READING: Section 3.3 says the backward products run in 16-bit precision; this oracle evaluates
them exactly in binary64 from the stored codes and scales, and the CUDA path is held to a tolerance
that covers its 16-bit operands (see tests/test_gpu_backward.py).  Pins: tests/test_oracle_backward.py
(adjoint identity of IHT against the forward rotation, finite differences of the linear forward map,
mask semantics, hand-computed 2 x 2 case).
"""
from __future__ import annotations

import numpy as np

from .definition import hadamard_matrix


def _container_bits(bits: int) -> int:
    return 1 if bits == 1 else 2 if bits == 2 else 4 if bits <= 4 else 8


def grid_values(codes: np.ndarray, cols: int, bits: int) -> np.ndarray:
    """Packed level indices -> c = 2k - (2^b - 1) as float64 [rows, cols] (element 0 in the low bits)."""
    cb = _container_bits(bits)
    per = 8 // cb
    codes = np.asarray(codes, dtype=np.uint8)
    shifts = (np.arange(per) * cb).astype(np.uint8)
    k = ((codes[:, :, None] >> shifts[None, None, :]) & ((1 << cb) - 1)).reshape(codes.shape[0], -1)[:, :cols]
    return 2.0 * k.astype(np.float64) - (2 ** bits - 1)


def mask_bits(mask: np.ndarray, cols: int) -> np.ndarray:
    """Trust-mask bitmap -> float64 0/1 [rows, cols] (element e at bit e mod 8 of byte e / 8)."""
    return np.unpackbits(np.asarray(mask, np.uint8), axis=1, bitorder="little")[:, :cols].astype(np.float64)


def iht(v: np.ndarray, g: int) -> np.ndarray:
    """Inverse orthonormal block Hadamard transform of each row (binary64)."""
    v = np.asarray(v, dtype=np.float64)
    rows, d = v.shape
    assert d % g == 0
    H = hadamard_matrix(g).astype(np.float64)
    return (v.reshape(rows, d // g, g) @ H / np.sqrt(g)).reshape(rows, d)      # H symmetric: H^T = H


def backward(dy: np.ndarray, xq: np.ndarray, sx: np.ndarray, mx: np.ndarray,
             wq: np.ndarray, sw: np.ndarray, mw: np.ndarray, K: int, bits: int, had_block: int,
             rows_x=None, rows_w=None) -> dict:
    """Algorithm 2.  ``rows_x`` / ``rows_w`` restrict the returned rows of dL/dx / dL/dw (for sampled
    checks at full size); the contraction always runs over everything."""
    dy = np.asarray(dy, dtype=np.float64)
    M, N = dy.shape
    xh = np.asarray(sx, np.float64)[:, None] * grid_values(xq, K, bits)          # xq_h  [M, K]
    wh = np.asarray(sw, np.float64)[:, None] * grid_values(wq, K, bits)          # wq_h  [N, K]
    rx = np.arange(M) if rows_x is None else np.asarray(rows_x)
    rw = np.arange(N) if rows_w is None else np.asarray(rows_w)
    d_xh = dy[rx] @ wh                                                            # dL/dxq_h
    dx = iht(mask_bits(mx, K)[rx] * d_xh, had_block)                              # dL/dx
    d_wh = dy[:, rw].T @ xh                                                       # dL/dwq_h
    dw = iht(mask_bits(mw, K)[rw] * d_wh, had_block)                              # dL/dw
    return {"dx": dx, "dw": dw, "d_xh": d_xh, "d_wh": d_wh}
