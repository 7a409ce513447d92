"""Pins for the FP4 (E2M1) grid variant of the oracle (Section 4.4, "The FP4 Format"), CPU only."""
import numpy as np

from oracle import definition as df
from oracle import quest_oracle as qo


def test_grid_is_e2m1_scaled_to_unit_interval_and_T_is_its_largest_half_interval():
    g = df.fp4_grid()
    assert len(g) == 15 and g[0] == -1.0 and g[-1] == 1.0 and g[7] == 0.0
    assert np.allclose(g[8:] * 6, [0.5, 1, 1.5, 2, 3, 4, 6]) and np.allclose(g, -g[::-1])
    # every positive E2M1 value is (1 + m/2) 2^(e-1) for e = 1..3, or m/2 for the subnormal row
    vals = sorted({(1 + m / 2) * 2.0 ** (e - 1) for e in (1, 2, 3) for m in (0, 1)} | {0.0, 0.5})
    assert np.allclose(g[7:] * 6, vals)
    assert np.isclose(np.max(np.diff(g * 6)) / 2, 1.0)          # largest half-interval on the value axis


def test_alpha_star_fp4_minimises_the_gaussian_mse_and_fp4_fits_worse_than_int4():
    pts = df.fp4_grid()
    lo, hi = 0.5, 8.0
    for _ in range(7):
        a = np.linspace(lo, hi, 2001)
        m = np.array([df.gaussian_mse_points(float(v), pts) for v in a])
        i = int(np.argmin(m))
        lo, hi = a[max(i - 2, 0)], a[min(i + 2, len(a) - 1)]
    a_tab = qo.alpha_star_fp4()
    assert abs(a_tab - a[i]) < 3e-5
    assert df.gaussian_mse_points(a_tab, pts) - m[i] < 1e-11
    # the general-grid closed form reproduces the uniform-grid one
    assert np.isclose(df.gaussian_mse_points(2.5140045, df.grid(4)), df.gaussian_mse(2.5140045, 4), rtol=1e-12)
    # the paper: with clipping allowed, FP4 has higher MSE than INT4 on Gaussian data
    assert df.gaussian_mse_points(a_tab, pts) > df.gaussian_mse(qo.alpha_star(4), 4)
    # quadrature of the quantiser itself
    xi = np.linspace(-12, 12, 1_200_001)
    q = a_tab * pts[np.argmin(np.abs((np.clip(xi, -a_tab, a_tab) / a_tab)[:, None] - pts[None, :]), axis=1)]
    quad = np.trapezoid((xi - q) ** 2 * np.exp(-0.5 * xi * xi) / np.sqrt(2 * np.pi), xi)
    assert abs(quad - df.gaussian_mse_points(a_tab, pts)) < 1e-7


def _values(codes, cols):
    return qo.unpack_fp4_twice(codes, cols).astype(np.float64) / 2.0


def test_codes_are_the_nearest_grid_points_of_the_definition():
    rng = np.random.default_rng(0)
    x = rng.standard_normal((64, 512)).astype(np.float32)
    x[rng.random(x.shape) < 0.01] *= 20
    for g in (1, 128, 512):
        out = qo.quantize_fp4(x, g, debug=True)
        ref = df.project_fp4(df.rotate(x, g), qo.alpha_star_fp4())
        v = _values(out["codes"], 512)
        clear = ref["margin"] > 1e-4
        assert clear.mean() > 0.999
        assert np.array_equal(v[clear], ref["v"][clear])
        assert np.allclose(out["scales"], ref["scale"], rtol=2e-6)
        # dequantised values are grid members and idempotent at fixed scale
        assert set(np.unique(np.abs(v))) <= {0, 0.5, 1, 1.5, 2, 3, 4, 6}


def test_ties_go_to_the_even_code_and_values_saturate():
    mags = [0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0]
    val = lambda code: (-1.0 if code & 8 else 1.0) * mags[code & 7]
    ties = {0.25: 0.0, 0.75: 1.0, 1.25: 1.0, 1.75: 2.0, 2.5: 2.0, 3.5: 4.0, 5.0: 4.0}      # the even code wins
    for t, want in ties.items():
        assert val(qo.e2m1_code(t)) == want and val(qo.e2m1_code(-t)) == -want
        lo, hi = np.nextafter(np.float32(t), np.float32(0)), np.nextafter(np.float32(t), np.float32(9))
        below = max(m for m in mags if m < t)
        above = min(m for m in mags if m > t)
        assert val(qo.e2m1_code(float(lo))) == below and val(qo.e2m1_code(float(hi))) == above
    for t in (6.0, 7.0, 1e9, float("inf")):
        assert val(qo.e2m1_code(t)) == 6.0 and val(qo.e2m1_code(-t)) == -6.0
    assert qo.e2m1_code(0.0) == 0 and qo.e2m1_code(-0.0) == 8 and qo.e2m1_code(-0.1) == 8      # the sign is kept at zero
    # every representable value maps to itself
    for i, m in enumerate(mags):
        assert qo.e2m1_code(m) == i and qo.e2m1_code(-m) == (8 | i)


def test_trust_mask_is_the_inequality_with_T_equal_to_one_value_step():
    rng = np.random.default_rng(1)
    x = (rng.standard_t(3, size=(32, 256))).astype(np.float32)
    for s in (1.0, 0.5, 1.3):
        out = qo.quantize_fp4(x, 128, s, debug=True)
        t = out["t"].astype(np.float64)
        v = _values(out["codes"], 256)
        want = np.abs(t - v) <= s * 1.0
        got = np.unpackbits(out["mask"], axis=1, bitorder="little").astype(bool)
        far = np.abs(np.abs(t - v) - s) > 1e-5
        assert np.array_equal(got[far], want[far])
    # at s = 1 every element inside the grid range is trusted (half-intervals are at most 1)
    out = qo.quantize_fp4(x, 128, 1.0, debug=True)
    got = np.unpackbits(out["mask"], axis=1, bitorder="little").astype(bool)
    assert got[np.abs(out["t"]) <= 6.0].all() and not got[np.abs(out["t"]) > 7.001].any()


def test_contraction_is_four_times_the_value_product():
    rng = np.random.default_rng(2)
    x = rng.standard_normal((9, 64)).astype(np.float32)
    w = rng.standard_normal((7, 64)).astype(np.float32)
    qx, qw = qo.quantize_fp4(x, 64), qo.quantize_fp4(w, 64)
    acc4 = qo.gemm_acc_fp4(qx["codes"], qw["codes"], 64)
    vx, vw = _values(qx["codes"], 64), _values(qw["codes"], 64)
    assert np.array_equal(acc4, np.rint(4 * vx @ vw.T).astype(np.int32))
    y = qo.dequant_fp4(acc4, qx["scales"], qw["scales"])
    ref = df.rotate(x, 64) @ df.rotate(w, 64).T                 # = x w^T: the rotation is orthonormal
    assert np.linalg.norm(y - ref) / np.linalg.norm(ref) < 0.2
