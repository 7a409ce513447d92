"""Pins for alpha*(b) (Section 3.1): the frozen table against a brute-force 1-D minimisation of
the Gaussian quantisation MSE, the closed form at b=1, and a quadrature of the quantiser itself."""
import math
import os

import numpy as np
import pytest

from oracle import definition as df
from oracle import quest_oracle as qo

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def brute_force_alpha(bits):
    lo, hi = 0.05, 8.0
    for _ in range(6):                       # dense grid, then refine around the best point
        a = np.linspace(lo, hi, 2001)
        m = np.array([df.gaussian_mse(float(v), bits) for v in a])
        i = int(np.argmin(m))
        lo, hi = a[max(i - 2, 0)], a[min(i + 2, len(a) - 1)]
    return float(a[i]), float(m[i])


def quadrature_mse(alpha, bits):
    """Integrate (xi - q(xi))^2 phi(xi) numerically with q written as clip-then-round."""
    L1 = 2 ** bits - 1
    xi = np.linspace(-12, 12, 2_400_001)
    lev = np.clip(np.rint(np.clip(xi, -alpha, alpha) / alpha * (L1 / 2) + L1 / 2 - 1e-15), 0, L1)
    q = alpha * (2 * lev - L1) / L1
    f = (xi - q) ** 2 * np.exp(-0.5 * xi * xi) / math.sqrt(2 * math.pi)
    return float(np.trapezoid(f, xi))


@pytest.mark.parametrize("bits", range(1, 9))
def test_table_minimises_the_gaussian_mse(bits):
    a_tab = qo.alpha_star(bits)
    a_bf, m_bf = brute_force_alpha(bits)
    assert abs(a_tab - a_bf) < 2e-5 * max(1.0, a_bf) * (10 if bits >= 7 else 1)
    assert df.gaussian_mse(a_tab, bits) - m_bf < 1e-11
    # stationarity and convexity around the table value
    e = 1e-3
    assert df.gaussian_mse(a_tab - e, bits) > df.gaussian_mse(a_tab, bits) < df.gaussian_mse(a_tab + e, bits)


@pytest.mark.parametrize("bits,expected", [(2, 0.118846), (3, 0.0374397), (4, 0.0115429), (8, 8.7686e-5)])
def test_minimum_mse_values(bits, expected):
    assert abs(df.gaussian_mse(qo.alpha_star(bits), bits) / expected - 1) < 2e-5


@pytest.mark.parametrize("bits", [1, 2, 4])
def test_closed_form_mse_matches_quadrature(bits):
    a = qo.alpha_star(bits)
    assert abs(df.gaussian_mse(a, bits) - quadrature_mse(a, bits)) < 1e-7
    assert abs(df.gaussian_mse(0.7 * a, bits) - quadrature_mse(0.7 * a, bits)) < 1e-7


def test_one_bit_closed_form_from_golden():
    with open(os.path.join(GOLD, "alpha_star_closed_form.txt")) as f:
        rows = [l.split() for l in f if not l.startswith("#")]
    b, a, m = int(rows[0][0]), float(rows[0][1]), float(rows[0][2])
    assert b == 1 and abs(a - math.sqrt(2 / math.pi)) < 1e-15
    assert abs(qo.alpha_star(1) - a) < 6e-8
    assert abs(df.gaussian_mse(a, 1) - m) < 1e-12


def test_alpha_increases_with_bits_and_is_zero_outside():
    vals = [qo.alpha_star(b) for b in range(1, 9)]
    assert all(x < y for x, y in zip(vals, vals[1:]))
    assert qo.alpha_star(0) == 0.0 and qo.alpha_star(9) == 0.0
