"""Pins for the weight-only forward oracle (Section 4.5), CPU only."""
import numpy as np
import torch

from oracle import backward as ob
from oracle import definition as od
from oracle import quest_oracle as qo
from oracle import weight_only as wo


def test_bf16_rounding_matches_the_library_conversion_and_rounds_ties_to_even():
    rng = np.random.default_rng(0)
    v = (rng.standard_normal(20000) * np.exp(rng.uniform(-20, 20, 20000))).astype(np.float32)
    got = wo.f32_to_bf16_bits(v)
    ref = torch.from_numpy(v).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(got, ref)
    # 1 + 2^-8 lies half-way between 1 and 1 + 2^-7: goes to the even neighbour 1; 1 + 3 * 2^-8 goes up to 1 + 2^-6
    ties = np.array([1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, -(1.0 + 2.0 ** -8)], np.float32)
    assert list(wo.f32_to_bf16_bits(ties)) == [0x3F80, 0x3F82, 0xBF80]
    assert np.array_equal(wo.bf16_bits_to_f32(np.array([0x3F80, 0xC000], np.uint16)), np.array([1.0, -2.0], np.float32))


def test_rotation_of_unit_vectors_gives_signed_columns_of_the_hadamard_matrix():
    for g in (4, 16, 128):
        H = od.hadamard_matrix(g)
        inv = np.float32(1.0) / np.sqrt(np.float32(g))
        for j in (0, 1, g - 1):
            x = np.zeros((1, g), np.float32)
            x[0, j] = 3.0
            xh = wo.bf16_bits_to_f32(wo.rotate_bf16(x, g))[0]
            expect = wo.bf16_bits_to_f32(wo.f32_to_bf16_bits(np.float32(3.0) * inv * H[j].astype(np.float32)))
            assert np.array_equal(xh, expect)
    # g = 4: 1 / sqrt(4) = 0.5 exactly
    x = np.array([[1.0, 2.0, 3.0, 4.0]], np.float32)
    assert np.array_equal(wo.bf16_bits_to_f32(wo.rotate_bf16(x, 4))[0], np.array([5.0, -1.0, -2.0, 0.0], np.float32))


def test_rotation_agrees_with_the_matrix_definition_to_bfloat16_rounding():
    rng = np.random.default_rng(1)
    for g, K in ((32, 64), (128, 256), (512, 512)):
        x = rng.standard_normal((6, K)).astype(np.float32)
        ref = od.rotate(x.astype(np.float64), g)                        # H_g / sqrt(g) blockwise, binary64
        got = wo.bf16_bits_to_f32(wo.rotate_bf16(x, g)).astype(np.float64)
        assert np.all(np.abs(got - ref) <= 2.0 ** -8 * np.abs(ref) + 1e-5)
        # bfloat16 input bits give the same result as the same values held in binary32
        xb = wo.f32_to_bf16_bits(x)
        assert np.array_equal(wo.rotate_bf16(xb, g), wo.rotate_bf16(wo.bf16_bits_to_f32(xb), g))


def test_output_equals_x_times_the_dequantised_weights_in_the_original_basis():
    # g = 16 and small-integer x: u is an integer below 2^8 and 1 / sqrt(16) = 1/4, so x_h is exact in
    # bfloat16 and y must equal x (IHT(w_q_h))^T, the plain definition of a linear layer with quantized weights.
    rng = np.random.default_rng(2)
    M, N, K, g = 9, 7, 64, 16
    x = rng.integers(-8, 9, size=(M, K)).astype(np.float32)
    w = (rng.standard_normal((N, K)) * 0.05).astype(np.float32)
    for bits in (1, 2, 3, 4, 8):
        out = wo.linear_fwd_weight_only(x, w, bits, g)
        assert np.array_equal(wo.bf16_bits_to_f32(out["xh"]).astype(np.float64), od.rotate(x.astype(np.float64), g))
        wq_h = ob.grid_values(out["wq"], K, bits) * out["sw"].astype(np.float64)[:, None]
        w_hat = ob.iht(wq_h, g)                                         # dequantised weights, original basis
        ref = x.astype(np.float64) @ w_hat.T
        assert np.allclose(out["y"], ref, rtol=1e-12, atol=1e-12)
        assert np.all(np.abs(out["y"]) <= out["bound"] + 1e-12)


def test_weight_outputs_are_those_of_the_quantizer_and_y_tracks_the_unquantized_layer():
    rng = np.random.default_rng(3)
    M, N, K, g = 16, 12, 256, 128
    x = rng.standard_normal((M, K)).astype(np.float32)
    w = (rng.standard_normal((N, K)) * 0.02).astype(np.float32)
    exact = x.astype(np.float64) @ w.astype(np.float64).T
    errs = []
    for bits in (2, 4, 8):
        out = wo.linear_fwd_weight_only(x, w, bits, g)
        q = qo.quantize(w, bits, g)
        assert np.array_equal(out["wq"], q["codes"]) and np.array_equal(out["sw"], q["scales"])
        assert np.array_equal(out["mw"], q["mask"])
        errs.append(np.linalg.norm(out["y"] - exact) / np.linalg.norm(exact))
    # relative error of the layer output falls with the weight width: about 0.34, 0.10, 0.01 for Gaussian weights
    assert errs[0] > errs[1] > errs[2]
    assert 0.2 < errs[0] < 0.5 and 0.05 < errs[1] < 0.2 and errs[2] < 0.03
