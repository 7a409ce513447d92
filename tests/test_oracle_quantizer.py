"""Pins for the projection (Eq. 1, Section 3.1) and the trust mask (Section 3.2) of the oracle."""
import math
import os

import numpy as np
import pytest

from oracle import definition as df
from oracle import quest_oracle as qo
from paper_2502_05003_b200 import synth
from tests.helpers import grid_values, unpack_levels, unpack_mask

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def make_rows(kind, rows, cols, seed):
    rng = np.random.default_rng(seed)
    if kind == "gauss":
        return rng.standard_normal((rows, cols)).astype(np.float32)
    if kind == "outliers":
        return synth.gaussian_with_outliers(rows, cols, rng)
    if kind == "student":
        return synth.student_t(rows, cols, rng)
    raise ValueError(kind)


@pytest.mark.parametrize("bits", [1, 2, 3, 4, 8])
@pytest.mark.parametrize("g,cols", [(1, 64), (8, 64), (128, 384), (512, 512)])
@pytest.mark.parametrize("kind", ["gauss", "outliers"])
def test_codes_are_the_nearest_grid_point(bits, g, cols, kind):
    """Exhaustive binary64 nearest-point search on the explicit grid of Eq. 1 gives the same
    level everywhere except within rounding noise of a cell boundary (then one level off)."""
    x = make_rows(kind, 24, cols, seed=bits * 1000 + g)
    out = qo.quantize(x, bits, g, debug=True)
    k = unpack_levels(out["codes"], cols, bits)
    ref = df.project(df.rotate(x, g), bits, qo.alpha_star(bits))
    diff = k != ref["k"]
    assert np.all(ref["margin"][diff] < 1e-4)
    assert np.all(np.abs(k - ref["k"])[diff] == 1)
    assert diff.mean() < 1e-3
    # scale: half step of the grid in the orthonormal Hadamard domain
    assert np.allclose(out["scales"], ref["scale"], rtol=2e-6, atol=0)
    # grid membership (golden Eq. 1 grid): xq / (alpha * rms) is an odd multiple of 1/(2^b-1)
    c = grid_values(k, bits)
    assert np.all(np.abs(c) <= 2 ** bits - 1) and np.all(c % 2 != 0)


def test_grid_matches_paper_fixture():
    with open(os.path.join(GOLD, "eq1_grid.txt")) as f:
        for line in f:
            if line.startswith("#"):
                continue
            parts = [int(v) for v in line.split()]
            b, nums = parts[0], parts[1:]
            assert len(nums) == 2 ** b and 0 not in nums
            assert np.allclose(df.grid(b), np.array(nums) / (2 ** b - 1))
            # the oracle reaches every grid point and no other: a cubic ramp spans +-2.6 RMS
            cols = 4096
            x = (np.linspace(-1, 1, cols) ** 3).astype(np.float32)[None, :]
            k = unpack_levels(qo.quantize(x, b, 1)["codes"], cols, b)
            assert sorted(set(grid_values(k, b).ravel().tolist())) == nums


@pytest.mark.parametrize("bits", [1, 2, 3, 4, 8])
def test_levels_are_monotone_in_the_rotated_value(bits):
    x = make_rows("student", 8, 1024, seed=bits)
    out = qo.quantize(x, bits, 128, debug=True)
    k = unpack_levels(out["codes"], 1024, bits)
    for r in range(8):
        order = np.argsort(out["u"][r], kind="stable")
        assert np.all(np.diff(k[r][order]) >= 0)
        assert k[r].min() == 0 and k[r].max() == 2 ** bits - 1 or bits == 8


@pytest.mark.parametrize("bits", [1, 2, 4, 8])
def test_sign_symmetry_and_power_of_two_scale_invariance(bits):
    x = make_rows("outliers", 6, 512, seed=11)
    a = qo.quantize(x, bits, 128, debug=True)
    b = qo.quantize(-x, bits, 128, debug=True)
    ka, kb = unpack_levels(a["codes"], 512, bits), unpack_levels(b["codes"], 512, bits)
    frac = np.abs(a["t"] - np.rint(a["t"]))
    off_tie = np.abs(frac - 0.5) > 1e-6
    assert np.array_equal(kb[off_tie], (2 ** bits - 1 - ka)[off_tie])
    assert np.array_equal(a["mask"], b["mask"])
    for m in (-20, 3, 40):
        s = qo.quantize(x * np.float32(2.0 ** m), bits, 128)
        assert np.array_equal(s["codes"], a["codes"]) and np.array_equal(s["mask"], a["mask"])
        assert np.array_equal(s["scales"], a["scales"] * np.float32(2.0 ** m))


def test_one_bit_is_the_sign_and_requantising_keeps_codes():
    x = make_rows("gauss", 4, 256, seed=5)
    out = qo.quantize(x, 1, 1, debug=True)
    k = unpack_levels(out["codes"], 256, 1)
    assert np.array_equal(k[x != 0], (x > 0).astype(np.int64)[x != 0])
    xq = out["scales"][:, None] * grid_values(k, 1)
    again = qo.quantize(xq.astype(np.float32), 1, 1)
    assert np.array_equal(again["codes"], out["codes"])
    # idempotence of the projection with the scale held fixed (every b): grid points map to themselves
    for bits in (2, 3, 4, 8):
        L1 = 2 ** bits - 1
        alpha = qo.alpha_star(bits)
        pts = alpha * df.grid(bits)
        lev = np.rint(np.clip(pts, -alpha, alpha) / alpha * (L1 / 2) + L1 / 2)
        assert np.array_equal(lev, np.arange(L1 + 1))


def test_zero_row_constant_row_and_single_outlier():
    x = np.zeros((3, 256), np.float32)
    x[1, :] = 3.0
    x[2, 17] = 1e6
    out = qo.quantize(x, 4, 128, trust_factor=1.0)
    k = unpack_levels(out["codes"], 256, 4)
    m = unpack_mask(out["mask"], 256)
    assert out["scales"][0] == 0.0 and np.all(k[0] == 8) and m[0].all()       # stated zero-row rule
    # a constant row concentrates in element 0 of each block: it is clipped high, the rest sit at 0
    assert np.all(k[1, [0, 128]] == 15) and np.all(np.delete(k[1], [0, 128]) == 8)
    assert not m[1, 0] and not m[1, 128] and np.delete(m[1], [0, 128]).all()
    # one spike becomes +-1e6 over its block and zero elsewhere: x_n = +-sqrt(2) in that block,
    # i.e. level rint(7.5 +- sqrt(2) * 15 / (2 alpha*)) = 12 or 3 (by hand)
    assert set(k[2, :128].tolist()) == {3, 12} and np.all(k[2, 128:] == 8)


def test_bf16_input_equals_widened_f32_input():
    x = make_rows("student", 16, 512, seed=9)
    bits16 = synth.f32_to_bf16_bits(x)
    a = qo.quantize(bits16, 4, 128)
    b = qo.quantize(synth.bf16_bits_to_f32(bits16), 4, 128)
    for key in ("codes", "scales", "mask"):
        assert np.array_equal(a[key], b[key])
    # the cast is round-to-nearest-even: error at most half a bfloat16 ulp
    assert np.max(np.abs(synth.bf16_bits_to_f32(bits16) - x) / np.abs(x)) <= 2.0 ** -8


def test_packing_layout_by_hand():
    """Element 0 of a byte sits in the low bits; mask bit e%8 of byte e//8."""
    # b=4, g=1: the first 8 elements sit mid-cell at known levels; 56 fillers bring the RMS to 1
    alpha, L1 = qo.alpha_star(4), 15
    want = np.array([0, 15, 1, 14, 7, 8, 3, 12])
    xn = (want - L1 / 2) / (L1 / 2) * alpha
    filler = math.sqrt((64 - float(np.sum(xn ** 2))) / 56)
    x = np.concatenate([xn, np.full(56, filler)])[None, :].astype(np.float32)
    out = qo.quantize(x, 4, 1)
    expect = [int(want[2 * i] | (want[2 * i + 1] << 4)) for i in range(4)]
    assert out["codes"][0, :4].tolist() == expect == [0xF0, 0xE1, 0x87, 0xC3]
    out2 = qo.quantize(x, 2, 1)          # b=2: four codes per byte
    k2 = unpack_levels(out2["codes"], 64, 2)[0]
    assert k2[:8].tolist() == [0, 3, 0, 3, 1, 2, 0, 3]
    assert out2["codes"][0, 0] == (k2[0] | k2[1] << 2 | k2[2] << 4 | k2[3] << 6)
    out1 = qo.quantize(x, 1, 1)          # b=1: eight per byte, same order as the mask bitmap
    k1 = unpack_levels(out1["codes"], 64, 1)[0]
    assert k1[:8].tolist() == [0, 1, 0, 1, 0, 1, 0, 1] and out1["codes"][0, 0] == 0xAA
    assert out1["codes"][0, 0] == sum(int(k1[i]) << i for i in range(8))
    out8 = qo.quantize(x, 8, 1)
    assert out8["codes"].shape == (1, 64)
    out3 = qo.quantize(x, 3, 1)          # b=3 lives in 4-bit containers
    assert out3["codes"].shape == (1, 32) and np.all(unpack_levels(out3["codes"], 64, 3) <= 7)


# ---------------------------------------------------------------- trust mask (Section 3.2)

@pytest.mark.parametrize("bits", [1, 2, 3, 4, 8])
@pytest.mark.parametrize("trust", [1.0, 1.3, 0.5])
def test_mask_is_the_inequality_in_binary64(bits, trust):
    x = make_rows("outliers", 16, 512, seed=bits)
    alpha = qo.alpha_star(bits)
    out = qo.quantize(x, bits, 128, trust_factor=trust, debug=True)
    m = unpack_mask(out["mask"], 512)
    k = unpack_levels(out["codes"], 512, bits)
    xh = df.rotate(x, 128)
    rms = np.sqrt(np.mean(xh ** 2, axis=1))
    xq = out["scales"].astype(np.float64)[:, None] * grid_values(k, bits)   # the oracle's own xq
    T = trust * alpha / (2 ** bits - 1) * rms[:, None]
    err = np.abs(xh - xq)
    ref = err <= T
    near = np.abs(err - T) < 2e-4 * T                     # ties and binary32 rounding noise
    assert np.array_equal(m[~near], ref[~near])
    assert near.mean() < 2e-3


@pytest.mark.parametrize("bits", [1, 2, 4, 8])
def test_unclipped_elements_are_always_trusted(bits):
    """For |x_n| <= alpha* the error is at most T (Section 3.2), so the bit is 1 at s >= 1."""
    x = make_rows("student", 16, 1024, seed=21)
    alpha = qo.alpha_star(bits)
    out = qo.quantize(x, bits, 128, trust_factor=1.0)
    m = unpack_mask(out["mask"], 1024)
    xh = df.rotate(x, 128)
    xn = xh / np.sqrt(np.mean(xh ** 2, axis=1, keepdims=True))
    assert m[np.abs(xn) <= alpha * (1 - 1e-6)].all()
    # and beyond alpha + T nothing is trusted
    assert not m[np.abs(xn) > (alpha + alpha / (2 ** bits - 1)) * (1 + 1e-6)].any()


def test_one_bit_trust_region_reaches_two_alpha():
    x = make_rows("gauss", 32, 1024, seed=2)
    alpha = qo.alpha_star(1)
    m = unpack_mask(qo.quantize(x, 1, 128, trust_factor=1.0)["mask"], 1024)
    xh = df.rotate(x, 128)
    xn = xh / np.sqrt(np.mean(xh ** 2, axis=1, keepdims=True))
    sure = np.abs(np.abs(xn) - 2 * alpha) > 1e-5
    assert np.array_equal(m[sure], (np.abs(xn) <= 2 * alpha)[sure])


@pytest.mark.parametrize("bits,trust,expected", [(1, 1.0, 0.1105), (2, 1.0, 0.04644), (3, 1.0, 0.01907),
                                                 (4, 1.0, 0.007327), (1, 1.3, 0.06649)])
def test_masked_fraction_on_gaussian_rows(bits, trust, expected):
    """With the rotation, the untrusted fraction is what a normal distribution predicts:
    2 (1 - Phi(alpha* + s T))."""
    alpha = qo.alpha_star(bits)
    closed = 2 * (1 - 0.5 * (1 + math.erf((alpha + trust * alpha / (2 ** bits - 1)) / math.sqrt(2))))
    assert abs(closed / expected - 1) < 2e-3
    x = make_rows("gauss", 128, 2048, seed=bits)
    m = unpack_mask(qo.quantize(x, bits, 128, trust_factor=trust)["mask"], 2048)
    n = m.size
    sigma = math.sqrt(closed * (1 - closed) / n)
    assert abs((1 - m.mean()) - closed) < 5 * sigma + 2e-4


def test_bad_arguments_are_rejected():
    x = np.zeros((2, 64), np.float32)
    for kw in (dict(bits=0), dict(bits=9), dict(had_block=3), dict(had_block=128), dict(trust_factor=-1.0),
               dict(trust_factor=float("nan"))):
        args = dict(bits=4, had_block=8, trust_factor=1.0)
        args.update(kw)
        with pytest.raises(ValueError):
            qo.quantize(x, args["bits"], args["had_block"], args["trust_factor"])
