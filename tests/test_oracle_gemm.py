"""Pins for the product step of Algorithm 1 in the oracle: the integer contraction and the scale product."""
import numpy as np
import pytest

from oracle import definition as df
from oracle import quest_oracle as qo
from paper_2502_05003_b200 import synth
from tests.helpers import container_bits, grid_values, unpack_levels


def pack_levels(levels, bits):
    cb = container_bits(bits)
    per = 8 // cb
    rows, cols = levels.shape
    out = np.zeros((rows, cols // per), np.uint8)
    for e in range(per):
        out |= (levels[:, e::per].astype(np.uint8) << (e * cb)).astype(np.uint8)
    return out


@pytest.mark.parametrize("bx,bw", [(4, 4), (1, 1), (2, 2), (3, 3), (8, 8), (4, 8), (1, 4)])
def test_acc_equals_int64_matmul_of_grid_values(bx, bw):
    rng = np.random.default_rng(bx * 10 + bw)
    M, N, K = 37, 29, 256
    kx = rng.integers(0, 2 ** bx, size=(M, K))
    kw = rng.integers(0, 2 ** bw, size=(N, K))
    acc = qo.gemm_acc(pack_levels(kx, bx), bx, pack_levels(kw, bw), bw, K)
    ref = grid_values(kx, bx) @ grid_values(kw, bw).T
    assert acc.dtype == np.int32 and np.array_equal(acc.astype(np.int64), ref)
    # brute-force triple loop on a corner
    cx, cw = grid_values(kx, bx), grid_values(kw, bw)
    for i in (0, M - 1):
        for j in (0, N - 1):
            assert acc[i, j] == sum(int(cx[i, k]) * int(cw[j, k]) for k in range(K))
    # every product of odd numbers is odd: parity of acc equals parity of K
    assert np.all((acc & 1) == (K & 1))


def test_special_cases():
    # identical one-hot-like rows: all levels at the top -> acc = K * (L-1)^2
    K = 64
    top = np.full((2, K), 15)
    acc = qo.gemm_acc(pack_levels(top, 4), 4, pack_levels(top, 4), 4, K)
    assert np.all(acc == K * 225)
    bot = np.zeros((3, K), np.int64)
    acc = qo.gemm_acc(pack_levels(top, 4), 4, pack_levels(bot, 4), 4, K)
    assert acc.shape == (2, 3) and np.all(acc == -K * 225)
    # K = 8 (smallest packed row), 1-bit: acc = K - 2 * hamming distance
    a = np.array([[1, 0, 1, 1, 0, 0, 1, 0]])
    b = np.array([[1, 1, 1, 0, 0, 0, 0, 0]])
    assert qo.gemm_acc(pack_levels(a, 1), 1, pack_levels(b, 1), 1, 8)[0, 0] == 8 - 2 * 3


def test_overflow_is_reported():
    K = 40000
    top = np.full((1, K), 255)
    with pytest.raises(ValueError):
        qo.gemm_acc(pack_levels(top, 8), 8, pack_levels(top, 8), 8, K)


def test_dequant_is_the_scale_product():
    rng = np.random.default_rng(0)
    acc = rng.integers(-10 ** 6, 10 ** 6, size=(5, 7)).astype(np.int32)
    sx = rng.random(5).astype(np.float32)
    sw = rng.random(7).astype(np.float32)
    y = qo.dequant(acc, sx, sw)
    assert np.allclose(y, sx.astype(np.float64)[:, None] * sw.astype(np.float64)[None, :] * acc, rtol=1e-15)


def test_linear_fwd_composes_the_steps():
    c = synth.config1()
    x, w = c["x"][:64], c["w"][:48]
    out = qo.linear_fwd(x, w, 4, 512, 1.0)
    qx, qw = qo.quantize(x, 4, 512), qo.quantize(w, 4, 512)
    assert np.array_equal(out["xq"], qx["codes"]) and np.array_equal(out["wq"], qw["codes"])
    assert np.array_equal(out["mx"], qx["mask"]) and np.array_equal(out["mw"], qw["mask"])
    cx = grid_values(unpack_levels(qx["codes"], 512, 4), 4)
    cw = grid_values(unpack_levels(qw["codes"], 512, 4), 4)
    assert np.array_equal(out["acc"], cx @ cw.T)
    y = (qx["scales"].astype(np.float64)[:, None] * cx) @ (qw["scales"].astype(np.float64)[:, None] * cw).T
    assert np.allclose(out["y"], y, rtol=1e-12, atol=1e-12)


def test_output_approximates_the_full_precision_product():
    """Identical rotations on both operands cancel (the transform is unitary): y ~ x w^T with
    no inverse transform, and the error shrinks as b grows."""
    rng = np.random.default_rng(4)
    x = rng.standard_normal((96, 512)).astype(np.float32)
    w = (rng.standard_normal((80, 512)) * 0.02).astype(np.float32)
    exact = x.astype(np.float64) @ w.astype(np.float64).T
    errs = []
    for bits in (1, 2, 3, 4, 8):
        y = qo.linear_fwd(x, w, bits, 128)["y"]
        errs.append(np.linalg.norm(y - exact) / np.linalg.norm(exact))
    assert all(a > b for a, b in zip(errs, errs[1:])), errs
    assert errs[-1] < 0.02 and errs[3] < 0.2
    # and the quantised product is exactly the product of the dequantised rotated operands
    out = qo.linear_fwd(x, w, 4, 128)
    xq = out["sx"].astype(np.float64)[:, None] * grid_values(unpack_levels(out["xq"], 512, 4), 4)
    wq = out["sw"].astype(np.float64)[:, None] * grid_values(unpack_levels(out["wq"], 512, 4), 4)
    assert np.allclose(out["y"], xq @ wq.T, rtol=1e-12, atol=1e-14)
    assert np.linalg.norm(xq - df.rotate(x, 128)) / np.linalg.norm(x) < 0.12
