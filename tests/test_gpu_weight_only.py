"""GPU parity: quest_linear_fwd_weight_only (Section 4.5) through the C ABI against the oracle.

Bit-exact: the rotated activations x_h (bfloat16), the weight codes, scales and trust masks.
The output sums K products of two exactly represented operands in binary32 on the tensor cores, in
an order (and with an alignment of addends) the hardware chooses: each of the K additions loses at
most one unit in the last place of the running sum, whose magnitude is at most
B = sw[n] sum_k |x_h c_w|, so  |y - y_exact| <= K 2^-23 B  elementwise (worst case; a random walk gives
about sqrt(K) 2^-24 B), plus 2^-8 |y| when y is stored as bfloat16.  The tests also require the
aggregate relative error of binary32 outputs to stay below 1e-5.
"""
import numpy as np
import pytest
import torch

from oracle import weight_only as wo
from paper_2502_05003_b200 import synth
from tests.gpu_util import to_dev

pytestmark = pytest.mark.gpu


def run_case(x_np, w_np, bits, g, trust=1.0, out_dtype=torch.float32, ldx=None):
    import paper_2502_05003_b200 as quest
    M, K = x_np.shape
    N = w_np.shape[0]
    xd = to_dev(x_np)
    if ldx is not None:                                   # rows of x inside a wider buffer
        wide = torch.zeros((M, ldx), dtype=xd.dtype, device="cuda")
        wide[:, :K] = xd
        xd = wide[:, :K]
    out = quest.quest_linear_fwd_weight_only(xd, to_dev(w_np), bits, g, trust, out_dtype=out_dtype)
    torch.cuda.synchronize()
    assert quest.quest_device_status() == 0
    ref = wo.linear_fwd_weight_only(x_np, w_np, bits, g, trust)
    assert np.array_equal(out["xh"].view(torch.int16).cpu().numpy().view(np.uint16), ref["xh"]), "x_h differs"
    assert np.array_equal(out["wq"].cpu().numpy(), ref["wq"]), "weight codes differ"
    assert np.array_equal(out["sw"].cpu().numpy(), ref["sw"]), "weight scales differ"
    assert np.array_equal(out["mw"].cpu().numpy(), ref["mw"]), "weight masks differ"
    got = out["y"].float().cpu().numpy().astype(np.float64)
    lim = K * 2.0 ** -23 * ref["bound"] + (2.0 ** -8 * np.abs(ref["y"]) if out_dtype == torch.bfloat16 else 0.0)
    err = np.abs(got - ref["y"])
    assert np.all(err <= lim + 1e-30), f"worst element at {np.max(err / (lim + 1e-30)):.3f} of the bound"
    rel = np.linalg.norm(got - ref["y"]) / max(np.linalg.norm(ref["y"]), 1e-30)
    assert rel < (4e-3 if out_dtype == torch.bfloat16 else 1e-5), f"relative error {rel:.2e}"
    return out


def gauss(rows, cols, seed, std=1.0, bf16=True):
    a = (np.random.default_rng(seed).standard_normal((rows, cols)) * std).astype(np.float32)
    return synth.f32_to_bf16_bits(a) if bf16 else a


@pytest.mark.parametrize("bits", [1, 2, 3, 4, 8])
def test_weight_widths_of_the_paper_and_eight_bits(bits):
    run_case(gauss(300, 256, 1), gauss(200, 256, 2, 0.02), bits, 128)


@pytest.mark.parametrize("M,N,K,g", [(1, 8, 32, 32), (37, 50, 96, 32), (130, 72, 128, 64), (129, 129, 512, 512),
                                     (64, 300, 2048, 2048), (520, 264, 4096, 4096), (257, 513, 1024, 128)])
def test_tile_edges_ragged_shapes_and_block_sizes(M, N, K, g):
    run_case(gauss(M, K, 3), gauss(N, K, 4, 0.02), 4, g)


def test_binary32_inputs_bfloat16_output_and_strided_rows():
    run_case(gauss(260, 384, 5, bf16=False), gauss(136, 384, 6, 0.02, bf16=False), 2, 128, out_dtype=torch.bfloat16)
    run_case(gauss(140, 256, 7), gauss(264, 256, 8, 0.02, bf16=False), 3, 128, ldx=320)


def test_heavy_tailed_activations_and_trust_factor():
    rng = np.random.default_rng(9)
    x = synth.f32_to_bf16_bits(synth.gaussian_with_outliers(384, 1024, rng))
    run_case(x, gauss(256, 1024, 10, 0.02), 4, 128, trust=0.5)
    run_case(x, gauss(256, 1024, 10, 0.02), 1, 128, trust=2.0)


def test_full_size_layer_in_the_benchmark_configuration():
    c = synth.config2()
    run_case(c["x"], c["w"], 4, 128, out_dtype=torch.bfloat16)


def test_empty_and_rejected_arguments():
    import paper_2502_05003_b200 as quest
    w = to_dev(gauss(16, 64, 11, 0.02))
    out = quest.quest_linear_fwd_weight_only(torch.empty((0, 64), dtype=torch.bfloat16, device="cuda"), w, 4, 32)
    assert out["y"].shape == (0, 16)
    x = to_dev(gauss(8, 64, 12))
    with pytest.raises(quest.QuestError) as e:
        quest.quest_linear_fwd_weight_only(x, w, 9, 32)
    assert e.value.status == 3
    with pytest.raises(quest.QuestError) as e:
        quest.quest_linear_fwd_weight_only(x, w, 4, 48)
    assert e.value.status == 4
    with pytest.raises(quest.QuestError) as e:
        quest.quest_linear_fwd_weight_only(x, w, 4, 32, workspace=torch.empty(256, dtype=torch.uint8, device="cuda"))
    assert e.value.status == 8
    with pytest.raises((quest.QuestError, ValueError)):
        quest.quest_linear_fwd_weight_only(to_dev(gauss(8, 48, 13)), to_dev(gauss(16, 48, 14)), 4, 16)
    assert quest.quest_weight_only_workspace_bytes(8, 16, 48) == 0
    assert quest.quest_weight_only_workspace_bytes(8, 16, 32768) == 0
