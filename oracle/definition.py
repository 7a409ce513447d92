"""The QuEST projection written out from its definition, in binary64 numpy.

TEST INFRASTRUCTURE ONLY.  This is the slowest, most literal form: an explicit Hadamard
matrix product, the RMS, and the projection of Section 3.1 evaluated exactly as the formula
reads (normalise, clip, round to the nearest grid point of Eq. 1, rescale).  It exists to pin
the canonical binary32 oracle in ``quest_oracle.c``: the two may disagree only where the
binary64 position is within rounding noise of a cell boundary.
"""
from __future__ import annotations

import numpy as np


def hadamard_matrix(g: int) -> np.ndarray:
    """Sylvester-Hadamard matrix, H[i, j] = (-1)^popcount(i & j), entries +-1 (int64)."""
    assert g >= 1 and g & (g - 1) == 0
    idx = np.arange(g)
    anded = idx[:, None] & idx[None, :]
    pop = np.zeros_like(anded)
    for bit in range(max(1, g.bit_length())):
        pop += (anded >> bit) & 1
    return 1 - 2 * (pop & 1)


def rotate(x: np.ndarray, g: int) -> np.ndarray:
    """Orthonormal block Hadamard transform of each row (Eq. 2's HT), binary64."""
    x = np.asarray(x, dtype=np.float64)
    rows, d = x.shape
    assert d % g == 0
    H = hadamard_matrix(g).astype(np.float64)
    xb = x.reshape(rows, d // g, g)
    return (xb @ H.T / np.sqrt(g)).reshape(rows, d)


def grid(bits: int) -> np.ndarray:
    """The 2^b points of Eq. 1's grid on [-1, 1]: odd multiples of 1/(2^b - 1)."""
    L1 = 2 ** bits - 1
    return (2 * np.arange(L1 + 1) - L1) / L1


def project(xh: np.ndarray, bits: int, alpha: float) -> dict:
    """proj_alpha(x_h) of Section 3.1 by exhaustive nearest-grid-point search (binary64).

    Returns level index ``k``, the projected values ``xq``, the per-row half step ``scale``
    (xq = scale * (2k - (2^b-1))) and the distance of each element to the nearest cell
    boundary on the level axis (``margin``; small margin = ambiguous rounding).
    """
    xh = np.asarray(xh, dtype=np.float64)
    L1 = 2 ** bits - 1
    rms = np.sqrt(np.mean(xh * xh, axis=1, keepdims=True))
    safe = np.where(rms > 0, rms, 1.0)
    xn = xh / safe                                      # RMS normalisation
    clipped = np.clip(xn, -alpha, alpha) / alpha        # clip(x, alpha) / alpha in [-1, 1]
    pts = grid(bits)
    dist = np.abs(clipped[..., None] - pts[None, None, :])
    k = np.argmin(dist, axis=-1)                        # nearest grid point (first on ties)
    xq = alpha * rms * pts[k]
    t = clipped * (L1 / 2.0) + L1 / 2.0                 # position on the level axis
    margin = np.abs((t - np.floor(t)) - 0.5)
    margin = np.where((t <= 0) | (t >= L1), 0.5, margin)
    return {"k": k, "xq": xq, "scale": (alpha * rms / L1)[:, 0], "rms": rms[:, 0],
            "margin": margin, "xn": xn}


def trust_mask(xh: np.ndarray, xq: np.ndarray, rms: np.ndarray, bits: int, alpha: float,
               trust_factor: float) -> np.ndarray:
    """M = [ |x_h - xq_h| <= T ], T = trust_factor * alpha / (2^b - 1) in RMS units (Sec. 3.2)."""
    T = trust_factor * alpha / (2 ** bits - 1) * rms[:, None]
    return np.abs(np.asarray(xh, np.float64) - xq) <= T


def gaussian_mse(alpha: float, bits: int) -> float:
    """E (xi - alpha*round(clip(xi, alpha)/alpha))^2 for xi ~ N(0,1) in closed form.

    Sum over the 2^b cells [lo, hi) of the integral of (xi - c)^2 phi(xi), using
    int phi = Phi, int xi phi = -phi, int xi^2 phi = Phi - xi phi.
    """
    from math import erf, exp, pi, sqrt, inf

    def Phi(v):
        return 0.5 * (1.0 + erf(v / sqrt(2.0)))

    def phi(v):
        return 0.0 if v in (inf, -inf) else exp(-0.5 * v * v) / sqrt(2.0 * pi)

    def xphi(v):
        return 0.0 if v in (inf, -inf) else v * phi(v)

    L1 = 2 ** bits - 1
    pts = [alpha * (2 * k - L1) / L1 for k in range(L1 + 1)]
    edges = [-inf] + [(pts[i] + pts[i + 1]) / 2 for i in range(L1)] + [inf]
    total = 0.0
    for k, c in enumerate(pts):
        lo, hi = edges[k], edges[k + 1]
        dPhi = Phi(hi) - Phi(lo)
        total += (dPhi - (xphi(hi) - xphi(lo))) + 2.0 * c * (phi(hi) - phi(lo)) + c * c * dPhi
    return total


# ---- FP4 (E2M1) grid of Section 4.4 "The FP4 Format" -------------------------------------------

E2M1_MAGNITUDES = (0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0)      # code magnitude index 0..7


def fp4_grid() -> np.ndarray:
    """The FP4 (E2M1) grid scaled to fit [-1, 1]: the 15 distinct values +-{0, .5, 1, 1.5, 2, 3, 4, 6} / 6."""
    m = np.array(E2M1_MAGNITUDES[1:]) / 6.0
    return np.concatenate([-m[::-1], [0.0], m])


def gaussian_mse_points(alpha: float, points) -> float:
    """E (xi - alpha * nearest(points, clip(xi, alpha) / alpha))^2 for xi ~ N(0,1), in closed form, for
    any sorted grid `points` on [-1, 1] whose end points are -1 and +1 (cells end at the midpoints)."""
    from math import erf, exp, pi, sqrt, inf

    def Phi(v):
        return 0.5 * (1.0 + erf(v / sqrt(2.0)))

    def phi(v):
        return 0.0 if v in (inf, -inf) else exp(-0.5 * v * v) / sqrt(2.0 * pi)

    def xphi(v):
        return 0.0 if v in (inf, -inf) else v * phi(v)

    pts = [alpha * float(p) for p in points]
    edges = [-inf] + [(pts[i] + pts[i + 1]) / 2 for i in range(len(pts) - 1)] + [inf]
    total = 0.0
    for k, c in enumerate(pts):
        lo, hi = edges[k], edges[k + 1]
        dPhi = Phi(hi) - Phi(lo)
        total += (dPhi - (xphi(hi) - xphi(lo))) + 2.0 * c * (phi(hi) - phi(lo)) + c * c * dPhi
    return total


def project_fp4(xh: np.ndarray, alpha: float) -> dict:
    """proj_alpha(x_h) with the FP4 grid by exhaustive nearest-point search (binary64).  Returns the
    projected values, the per-row scale (xq = scale * v with v the E2M1 value in [-6, 6]), the
    position t on the E2M1 value axis and the margin to the nearest cell boundary."""
    xh = np.asarray(xh, dtype=np.float64)
    rms = np.sqrt(np.mean(xh * xh, axis=1, keepdims=True))
    safe = np.where(rms > 0, rms, 1.0)
    clipped = np.clip(xh / safe, -alpha, alpha) / alpha
    pts = fp4_grid()
    k = np.argmin(np.abs(clipped[..., None] - pts[None, None, :]), axis=-1)
    t = clipped * 6.0
    vals = pts * 6.0
    edges = (vals[:-1] + vals[1:]) / 2
    margin = np.min(np.abs(t[..., None] - edges[None, None, :]), axis=-1)
    return {"v": vals[k], "xq": alpha * rms * pts[k], "scale": (alpha * rms / 6.0)[:, 0], "rms": rms[:, 0],
            "t": t, "margin": margin}
