"""Pins for the MLP-block oracle (gate / up / SwiGLU / down with QuEST linear layers), CPU only."""
import math

import numpy as np

from oracle import mlp
from oracle import quest_oracle as qo
from paper_2502_05003_b200 import synth


def test_silu_against_closed_forms_and_identities():
    # silu(0) = 0; silu(z) - silu(-z) = z (sigmoid(z) + sigmoid(-z) = 1); silu(ln 3) = ln 3 * 3/4
    assert mlp.silu(np.array([0.0]))[0] == 0.0
    z = np.linspace(-30, 30, 2001)
    assert np.allclose(mlp.silu(z) - mlp.silu(-z), z, rtol=0, atol=1e-13)
    assert abs(mlp.silu(np.array([math.log(3.0)]))[0] - math.log(3.0) * 0.75) < 1e-15
    assert abs(mlp.silu(np.array([-math.log(3.0)]))[0] + math.log(3.0) * 0.25) < 1e-15
    # large arguments neither overflow nor lose the tail: silu(z) -> z, silu(-z) -> -z exp(-z)
    assert mlp.silu(np.array([800.0]))[0] == 800.0
    assert mlp.silu(np.array([-800.0]))[0] == 0.0 or abs(mlp.silu(np.array([-800.0]))[0]) < 1e-300
    assert abs(mlp.silu(np.array([-40.0]))[0] / (-40.0 * math.exp(-40.0)) - 1.0) < 1e-12
    # against the textbook definition written independently with math.exp
    for v in (-7.3, -1.0, -1e-3, 1e-3, 0.5, 2.0, 11.0):
        assert abs(mlp.silu(np.array([v]))[0] - v / (1.0 + math.exp(-v))) <= 1e-15 * max(1.0, abs(v))
    # minimum of silu: z = -1.2784645..., value -0.2784645...
    zz = np.linspace(-2, 0, 200001)
    i = np.argmin(mlp.silu(zz))
    assert abs(zz[i] + 1.2784645) < 2e-5 and abs(mlp.silu(zz)[i] + 0.2784645) < 1e-7


def _tiny(seed=0, T=24, H=64, I=96):
    rng = np.random.default_rng(seed)
    x = synth.f32_to_bf16_bits(synth.student_t(T, H, rng))
    wg = synth.f32_to_bf16_bits(synth.weights(I, H, rng))
    wu = synth.f32_to_bf16_bits(synth.weights(I, H, rng))
    wd = synth.f32_to_bf16_bits(synth.weights(H, I, rng))
    return x, wg, wu, wd


def test_hidden_is_built_from_two_algorithm_1_layers_sharing_one_quantized_x():
    x, wg, wu, _ = _tiny()
    out = mlp.hidden(x, wg, wu, 4, 32)
    lg, lu = qo.linear_fwd(x, wg, 4, 32), qo.linear_fwd(x, wu, 4, 32)
    assert np.array_equal(out["x"]["codes"], lg["xq"]) and np.array_equal(out["x"]["codes"], lu["xq"])
    assert np.array_equal(out["gate"], lg["y"]) and np.array_equal(out["up"], lu["y"])
    # element by element, with the exponential written out again
    for (i, j) in ((0, 0), (5, 17), (23, 95)):
        g, u = lg["y"][i, j], lu["y"][i, j]
        assert abs(out["h"][i, j] - g / (1.0 + math.exp(-g)) * u) <= 1e-14 * abs(g * u) + 1e-300


def test_hidden_approaches_the_unquantized_block_as_bits_grow():
    x, wg, wu, _ = _tiny(1, T=32, H=128, I=64)
    xf = synth.bf16_bits_to_f32(x).astype(np.float64)
    g = xf @ synth.bf16_bits_to_f32(wg).astype(np.float64).T
    u = xf @ synth.bf16_bits_to_f32(wu).astype(np.float64).T
    exact = g / (1.0 + np.exp(-g)) * u
    errs = [np.linalg.norm(mlp.hidden(x, wg, wu, b, 128)["h"] - exact) / np.linalg.norm(exact) for b in (2, 4, 8)]
    assert errs[0] > errs[1] > errs[2] and errs[2] < 0.05


def test_sampled_rows_equal_the_full_computation():
    x, wg, wu, wd = _tiny(2)
    full = mlp.hidden(x, wg, wu, 4, 32)
    rows = [3, 11, 20]
    part = mlp.hidden(x, wg, wu, 4, 32, rows=rows)
    assert np.array_equal(part["h"], full["h"][rows])
    h16 = synth.f32_to_bf16_bits(full["h"].astype(np.float32))
    d_full = mlp.down_from_hidden(h16, wd, 4, 32)
    d_part = mlp.down_from_hidden(h16, wd, 4, 32, rows=rows)
    assert np.array_equal(d_part["y"], d_full["y"][rows])


def test_down_projection_is_algorithm_1_on_the_stored_hidden_activations():
    x, wg, wu, wd = _tiny(3)
    h16 = synth.f32_to_bf16_bits(mlp.hidden(x, wg, wu, 4, 32)["h"].astype(np.float32))
    d = mlp.down_from_hidden(h16, wd, 4, 32)
    ref = qo.linear_fwd(h16, wd, 4, 32)
    assert np.array_equal(d["y"], ref["y"]) and np.array_equal(d["h"]["codes"], ref["xq"])
    assert np.array_equal(d["h"]["mask"], ref["mx"]) and np.array_equal(d["w_down"]["codes"], ref["wq"])
