"""Pins for the rotation step (Eq. 2, "Hadamard Preprocessing"): the oracle's butterflies
against the explicit Sylvester matrix and the identities an orthogonal +-1 matrix obeys."""
import numpy as np
import pytest

from oracle import definition as df
from oracle import quest_oracle as qo


def test_h2_h4_by_hand():
    assert df.hadamard_matrix(2).tolist() == [[1, 1], [1, -1]]
    assert df.hadamard_matrix(4).tolist() == [[1, 1, 1, 1], [1, -1, 1, -1], [1, 1, -1, -1], [1, -1, -1, 1]]


@pytest.mark.parametrize("g", [1, 2, 8, 128, 512, 1024])
def test_h_ht_equals_g_identity(g):
    H = df.hadamard_matrix(g)
    assert np.array_equal(H @ H.T, g * np.eye(g, dtype=np.int64))
    assert np.array_equal(H, H.T)


@pytest.mark.parametrize("g", [2, 4, 16, 128, 2048])
def test_butterflies_on_unit_vectors_give_matrix_columns(g):
    H = df.hadamard_matrix(g)
    for j in list(range(min(g, 5))) + [g - 1, g // 2, g // 2 + 1 if g > 2 else 0]:
        e = np.zeros(g, np.float32)
        e[j] = 1.0
        assert np.array_equal(qo.fwht_block(e), H[:, j].astype(np.float32)), (g, j)


@pytest.mark.parametrize("g", [2, 8, 64, 128, 512, 4096])
def test_exact_on_small_integers(g):
    rng = np.random.default_rng(g)
    x = rng.integers(-7, 8, size=g).astype(np.float32)
    u = qo.fwht_block(x)
    H = df.hadamard_matrix(g)
    assert np.array_equal(u.astype(np.int64), H @ x.astype(np.int64))        # the definition
    assert np.array_equal(qo.fwht_block(u), np.float32(g) * x)                 # H H = g I
    assert int((u.astype(np.int64) ** 2).sum()) == g * int((x.astype(np.int64) ** 2).sum())  # Parseval


@pytest.mark.parametrize("g", [16, 128, 1024])
def test_close_to_matrix_product_on_floats(g):
    rng = np.random.default_rng(7)
    x = rng.standard_normal(g).astype(np.float32)
    u = qo.fwht_block(x)
    ref = df.hadamard_matrix(g).astype(np.float64) @ x.astype(np.float64)
    assert np.max(np.abs(u - ref)) <= 1e-5 * np.sqrt(g) * np.max(np.abs(ref))
    # norm preservation of the orthonormal transform
    assert abs(np.linalg.norm(u.astype(np.float64)) / np.sqrt(g) / np.linalg.norm(x.astype(np.float64)) - 1) < 1e-6


def test_block_diagonal_rotation_in_quantize():
    """The rotation inside quantize() acts per contiguous block of g along the row."""
    rng = np.random.default_rng(3)
    x = rng.standard_normal((5, 384)).astype(np.float32)
    out = qo.quantize(x, 4, 128, debug=True)
    for r in range(5):
        for blk in range(3):
            seg = x[r, blk * 128:(blk + 1) * 128]
            assert np.array_equal(out["u"][r, blk * 128:(blk + 1) * 128], qo.fwht_block(seg))
    ref = df.rotate(x, 128) * np.sqrt(128)
    assert np.allclose(out["u"], ref, rtol=0, atol=1e-4)
