"""GPU parity: quest_linear_bwd (Algorithm 2) through the C ABI against the binary64 oracle.

The CUDA path rounds one operand of every product to bfloat16 (the other, an integer grid value, is
exact) and accumulates in binary32, so each masked product-sum d[i][k] carries an absolute error of at
most 2^-9 * sum_n |term| (rounding of dy * scale) plus binary32 accumulation noise.  The inverse
Hadamard transform is orthonormal, so per output row  ||got - ref||_2 <= 2^-9 * ||B_row||_2  with
B[i][k] = sum_n |dy| |quantized operand|; the tests allow twice that (2^-8) and, for bfloat16 outputs,
add the storage rounding 2^-8 |ref|.
"""
import numpy as np
import pytest
import torch

from oracle import backward as ob
from oracle import quest_oracle as qo
from paper_2502_05003_b200 import synth
from tests.gpu_util import to_dev

pytestmark = pytest.mark.gpu

BOUND = 2.0 ** -8


def run_case(x_np, w_np, bits, g, seed=0, out_dtype=torch.float32, rows_x=None, rows_w=None):
    import paper_2502_05003_b200 as quest
    M, K = x_np.shape
    N = w_np.shape[0]
    fx, fw = qo.quantize(x_np, bits, g), qo.quantize(w_np, bits, g)
    rng = np.random.default_rng(seed)
    dy_bits = synth.f32_to_bf16_bits(rng.standard_normal((M, N)).astype(np.float32))
    dy64 = synth.bf16_bits_to_f32(dy_bits).astype(np.float64)
    fwd = {"xq": torch.from_numpy(fx["codes"]).cuda(), "sx": torch.from_numpy(fx["scales"]).cuda(),
           "mx": torch.from_numpy(fx["mask"]).cuda(), "wq": torch.from_numpy(fw["codes"]).cuda(),
           "sw": torch.from_numpy(fw["scales"]).cuda(), "mw": torch.from_numpy(fw["mask"]).cuda()}
    out = quest.quest_linear_bwd(to_dev(dy_bits), fwd, bits, g, K, out_dtype=out_dtype)
    torch.cuda.synchronize()
    assert quest.quest_device_status() == 0
    rx = np.arange(M) if rows_x is None else np.sort(np.asarray(rows_x))
    rw = np.arange(N) if rows_w is None else np.sort(np.asarray(rows_w))
    ref = ob.backward(dy64, fx["codes"], fx["scales"], fx["mask"], fw["codes"], fw["scales"], fw["mask"], K, bits, g,
                      rows_x=rx, rows_w=rw)
    xh = np.abs(fx["scales"].astype(np.float64)[:, None] * ob.grid_values(fx["codes"], K, bits))
    wh = np.abs(fw["scales"].astype(np.float64)[:, None] * ob.grid_values(fw["codes"], K, bits))
    bx = np.abs(dy64[rx]) @ wh                                 # [rows, K] sums of |terms|
    bw = np.abs(dy64[:, rw]).T @ xh
    for name, got_t, want, b, rows in (("dx", out["dx"], ref["dx"], bx, rx), ("dw", out["dw"], ref["dw"], bw, rw)):
        got = got_t.float().cpu().numpy().astype(np.float64)[rows]
        err = np.linalg.norm(got - want, axis=1)
        lim = BOUND * np.linalg.norm(b, axis=1) + (BOUND * np.linalg.norm(want, axis=1) if out_dtype == torch.bfloat16 else 0.0)
        assert np.all(err <= lim + 1e-30), f"{name}: worst row at {np.max(err / (lim + 1e-30)):.3f} of the bound"
        # and it is not merely inside a loose bound: the result is accurate to 16-bit operand precision
        rel = np.linalg.norm(got - want) / max(np.linalg.norm(want), 1e-30)
        assert rel < (8e-3 if out_dtype == torch.bfloat16 else 5e-3), f"{name}: relative error {rel:.2e}"
    return out


def gauss(rows, cols, seed, std=1.0, bf16=True):
    a = (np.random.default_rng(seed).standard_normal((rows, cols)) * std).astype(np.float32)
    return synth.f32_to_bf16_bits(a) if bf16 else a


@pytest.mark.parametrize("M,N,K", [(256, 192, 512), (8, 8, 32), (136, 264, 1024), (512, 128, 128), (40, 1000, 2048)])
def test_shapes(M, N, K):
    g = min(128, K)
    run_case(gauss(M, K, 1), gauss(N, K, 2, 0.02), 4, g, seed=M + N)


@pytest.mark.parametrize("bits", [1, 2, 3, 8])
def test_bit_widths(bits):
    run_case(gauss(264, 1024, 3), gauss(320, 1024, 4, 0.02), bits, 128, seed=bits)


@pytest.mark.parametrize("g", [1, 32, 512, 2048])
def test_hadamard_block_sizes(g):
    run_case(gauss(200, 2048, 5), gauss(256, 2048, 6, 0.02), 4, g, seed=g)


def test_bf16_outputs_and_single_gradients():
    import paper_2502_05003_b200 as quest
    x, w = gauss(256, 512, 7), gauss(384, 512, 8, 0.02)
    out = run_case(x, w, 4, 128, seed=9, out_dtype=torch.bfloat16)
    assert out["dx"].dtype == torch.bfloat16
    fx, fw = qo.quantize(x, 4, 128), qo.quantize(w, 4, 128)
    fwd = {k: torch.from_numpy(v).cuda() for k, v in (("xq", fx["codes"]), ("sx", fx["scales"]), ("mx", fx["mask"]),
                                                      ("wq", fw["codes"]), ("sw", fw["scales"]), ("mw", fw["mask"]))}
    dy = to_dev(synth.f32_to_bf16_bits(np.random.default_rng(9).standard_normal((256, 384)).astype(np.float32)))
    only_x = quest.quest_linear_bwd(dy, fwd, 4, 128, 512, out_dtype=torch.bfloat16, want_dw=False)
    only_w = quest.quest_linear_bwd(dy, fwd, 4, 128, 512, out_dtype=torch.bfloat16, want_dx=False)
    torch.cuda.synchronize()
    assert only_x["dw"] is None and only_w["dx"] is None
    assert torch.equal(only_x["dx"], out["dx"]) and torch.equal(only_w["dw"], out["dw"])


def test_forward_then_backward_on_the_gpu_outputs():
    """The backward call consumes exactly what quest_linear_fwd returned."""
    import paper_2502_05003_b200 as quest
    c = synth.config1()
    x, w = to_dev(c["x"]), to_dev(c["w"])
    fwd = quest.quest_linear_fwd(x, w, 4, 512, 1.0, out_dtype=torch.float32)
    dy_bits = synth.f32_to_bf16_bits(np.random.default_rng(0).standard_normal((256, 512)).astype(np.float32))
    out = quest.quest_linear_bwd(to_dev(dy_bits), fwd, 4, 512, 512)
    torch.cuda.synchronize()
    ref = ob.backward(synth.bf16_bits_to_f32(dy_bits), fwd["xq"].cpu().numpy(), fwd["sx"].cpu().numpy(),
                      fwd["mx"].cpu().numpy(), fwd["wq"].cpu().numpy(), fwd["sw"].cpu().numpy(), fwd["mw"].cpu().numpy(),
                      512, 4, 512)
    for k in ("dx", "dw"):
        got = out[k].cpu().numpy().astype(np.float64)
        assert np.linalg.norm(got - ref[k]) <= 5e-3 * np.linalg.norm(ref[k])


def test_config2_full_size_sampled_rows():
    c = synth.config2()
    rx = np.random.default_rng(0).choice(4096, 48, replace=False)
    rw = np.random.default_rng(1).choice(2048, 48, replace=False)
    run_case(c["x"], c["w"], 4, 128, seed=2, rows_x=rx, rows_w=rw)


def test_argument_errors():
    import paper_2502_05003_b200 as quest
    z = lambda *s, dt=torch.uint8: torch.zeros(s, dtype=dt, device="cuda")
    fwd = {"xq": z(16, 64), "sx": z(16, dt=torch.float32), "mx": z(16, 16), "wq": z(16, 64),
           "sw": z(16, dt=torch.float32), "mw": z(16, 16)}
    dy = z(16, 16, dt=torch.bfloat16)
    with pytest.raises(quest.QuestError):
        quest.quest_linear_bwd(dy, fwd, 0, 128, 128)
    with pytest.raises(quest.QuestError):
        quest.quest_linear_bwd(dy, fwd, 4, 96, 128)
    with pytest.raises(ValueError):
        quest.quest_linear_bwd(z(12, 16, dt=torch.bfloat16), fwd, 4, 128, 128)       # M not a multiple of 8
