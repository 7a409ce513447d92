"""Pins for the backward oracle (Algorithm 2), CPU only."""
import numpy as np

from oracle import backward as ob
from oracle import definition as od
from oracle import quest_oracle as qo


def _forward(M=24, N=16, K=256, bits=4, g=128, seed=0):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((M, K)).astype(np.float32)
    w = (rng.standard_normal((N, K)) * 0.05).astype(np.float32)
    fx, fw = qo.quantize(x, bits, g), qo.quantize(w, bits, g)
    return x, w, fx, fw


def test_iht_inverts_the_forward_rotation_and_is_its_adjoint():
    rng = np.random.default_rng(1)
    for g, d in ((1, 8), (2, 8), (8, 64), (128, 256), (256, 256)):
        v = rng.standard_normal((5, d))
        u = rng.standard_normal((5, d))
        assert np.allclose(ob.iht(od.rotate(v, g), g), v, atol=1e-12)            # IHT(HT(v)) = v
        assert np.allclose(np.sum(ob.iht(u, g) * v), np.sum(u * od.rotate(v, g)), atol=1e-10)   # <IHT u, v> = <u, HT v>
        assert np.allclose(np.sum(ob.iht(v, g) ** 2), np.sum(v ** 2))            # orthonormal


def test_two_by_two_case_by_hand():
    # g = 2, K = 2, b = 1: grid values +-1.  x codes (1, 0) -> c = (+1, -1); w codes (1, 1) -> (+1, +1).
    xq = np.array([[0b01]], np.uint8)        # element 0 = level 1, element 1 = level 0
    wq = np.array([[0b11]], np.uint8)
    sx, sw = np.array([2.0], np.float32), np.array([0.5], np.float32)
    ones = np.array([[0b11]], np.uint8)
    out = ob.backward(np.array([[3.0]]), xq, sx, ones, wq, sw, ones, K=2, bits=1, had_block=2)
    # dL/dxq_h = 3 * (0.5, 0.5) = (1.5, 1.5); IHT with H_2/sqrt(2): ((1.5 + 1.5), (1.5 - 1.5)) / sqrt(2)
    assert np.allclose(out["dx"], [[3.0 / np.sqrt(2.0), 0.0]])
    # dL/dwq_h = 3 * (2, -2) = (6, -6); IHT: (0, 12) / sqrt(2)
    assert np.allclose(out["dw"], [[0.0, 12.0 / np.sqrt(2.0)]])
    # masking element 1 of x: (1.5, 0) -> (1.5, 1.5) / sqrt(2)
    out2 = ob.backward(np.array([[3.0]]), xq, sx, np.array([[0b01]], np.uint8), wq, sw, ones, K=2, bits=1, had_block=2)
    assert np.allclose(out2["dx"], [[1.5 / np.sqrt(2.0), 1.5 / np.sqrt(2.0)]])


def test_gradients_match_finite_differences_of_the_linear_forward_map():
    """With the codes held fixed, y = xq_h wq_h^T is linear in xq_h and in wq_h, and x -> HT(x) is
    linear: for all-ones masks, dL/dx of L = <dy, HT(x) wq_h^T> is IHT(dy wq_h) exactly."""
    x, w, fx, fw = _forward()
    M, K = x.shape
    N = w.shape[0]
    g, bits = 128, 4
    rng = np.random.default_rng(2)
    dy = rng.standard_normal((M, N))
    ones_x = np.full((M, K // 8), 0xFF, np.uint8)
    ones_w = np.full((N, K // 8), 0xFF, np.uint8)
    out = ob.backward(dy, fx["codes"], fx["scales"], ones_x, fw["codes"], fw["scales"], ones_w, K, bits, g)
    wh = fw["scales"].astype(np.float64)[:, None] * ob.grid_values(fw["codes"], K, bits)
    xh = fx["scales"].astype(np.float64)[:, None] * ob.grid_values(fx["codes"], K, bits)
    L_x = lambda xx: np.sum(dy * (od.rotate(xx, g) @ wh.T))
    L_w = lambda ww: np.sum(dy * (xh @ od.rotate(ww, g).T))
    x64, w64 = x.astype(np.float64), w.astype(np.float64)
    for (i, j) in ((0, 0), (3, 17), (23, 255), (11, 128)):
        e = np.zeros_like(x64); e[i, j] = 1.0
        assert np.isclose(L_x(x64 + e) - L_x(x64), out["dx"][i, j], rtol=1e-9, atol=1e-9)
    for (i, j) in ((0, 0), (5, 100), (15, 255)):
        e = np.zeros_like(w64); e[i, j] = 1.0
        assert np.isclose(L_w(w64 + e) - L_w(w64), out["dw"][i, j], rtol=1e-9, atol=1e-9)


def test_masked_elements_pass_no_gradient_in_the_hadamard_domain():
    x, w, fx, fw = _forward(bits=2, seed=3)
    M, K = x.shape
    N = w.shape[0]
    dy = np.random.default_rng(4).standard_normal((M, N))
    out = ob.backward(dy, fx["codes"], fx["scales"], fx["mask"], fw["codes"], fw["scales"], fw["mask"], K, 2, 128)
    # HT(dL/dx) recovers M * dL/dxq_h: zero exactly where the forward mask is zero
    back = od.rotate(out["dx"], 128)
    mbits = ob.mask_bits(fx["mask"], K)
    assert (mbits == 0).any()
    assert np.allclose(back[mbits == 0], 0.0, atol=1e-10)
    assert np.allclose(back[mbits == 1], out["d_xh"][mbits == 1], atol=1e-9)
    zero = ob.backward(dy, fx["codes"], fx["scales"], np.zeros_like(fx["mask"]), fw["codes"], fw["scales"],
                       np.zeros_like(fw["mask"]), K, 2, 128)
    assert not zero["dx"].any() and not zero["dw"].any()


def test_row_subsets_equal_the_full_result():
    x, w, fx, fw = _forward(seed=5)
    M, K = x.shape
    N = w.shape[0]
    dy = np.random.default_rng(6).standard_normal((M, N))
    full = ob.backward(dy, fx["codes"], fx["scales"], fx["mask"], fw["codes"], fw["scales"], fw["mask"], K, 4, 128)
    part = ob.backward(dy, fx["codes"], fx["scales"], fx["mask"], fw["codes"], fw["scales"], fw["mask"], K, 4, 128,
                       rows_x=[1, 7, 20], rows_w=[0, 15])
    assert np.allclose(part["dx"], full["dx"][[1, 7, 20]]) and np.allclose(part["dw"], full["dw"][[0, 15]])
