"""GPU parity: quest_linear_fwd (Algorithm 1 end to end) on the benchmark configurations."""
import numpy as np
import pytest
import torch

from oracle import quest_oracle as qo
from paper_2502_05003_b200 import synth
from tests.gpu_util import BF16_OUT_RTOL, assert_output_close, to_dev

pytestmark = pytest.mark.gpu

F32_IN_RTOL = 1e-5                   # fp32 inputs, fp32 output
BF16_IN_RTOL = 2e-3                  # bf16 inputs, fp32 output


def check_linear(x_np, w_np, bits, g, trust, out_dtype, y_tol, sample_rows=None):
    import paper_2502_05003_b200 as quest
    x, w = to_dev(x_np), to_dev(w_np)
    out = quest.quest_linear_fwd(x, w, bits, g, trust, out_dtype=out_dtype)
    torch.cuda.synchronize()
    assert quest.quest_device_status() == 0
    qx, qw = qo.quantize(x_np, bits, g, trust), qo.quantize(w_np, bits, g, trust)
    assert np.array_equal(out["xq"].cpu().numpy(), qx["codes"])
    assert np.array_equal(out["wq"].cpu().numpy(), qw["codes"])
    assert np.array_equal(out["mx"].cpu().numpy(), qx["mask"])
    assert np.array_equal(out["mw"].cpu().numpy(), qw["mask"])
    assert np.allclose(out["sx"].cpu().numpy(), qx["scales"], rtol=1e-5, atol=0)
    assert np.allclose(out["sw"].cpu().numpy(), qw["scales"], rtol=1e-5, atol=0)
    rows = np.arange(x_np.shape[0]) if sample_rows is None else np.sort(np.asarray(sample_rows))
    K = x_np.shape[1]
    ref_y = qo.dequant(qo.gemm_acc(qx["codes"][rows], bits, qw["codes"], bits, K), qx["scales"][rows], qw["scales"])
    got = out["y"].float().cpu().numpy().astype(np.float64)[rows]
    if out_dtype == torch.bfloat16:
        assert_output_close(got, ref_y, True)
    else:
        assert np.all(np.abs(got - ref_y) <= y_tol * np.abs(ref_y) + 1e-30)
    if out_dtype == torch.bfloat16:
        # the same call with an fp32 result must meet the tolerance stated for bf16 inputs
        y32 = quest.quest_linear_fwd(x, w, bits, g, trust, out_dtype=torch.float32)["y"]
        got32 = y32.cpu().numpy().astype(np.float64)[rows]
        assert np.all(np.abs(got32 - ref_y) <= BF16_IN_RTOL * np.abs(ref_y) + 1e-30)
        assert np.all(np.abs(got32 - ref_y) <= F32_IN_RTOL * np.abs(ref_y) + 1e-30)
    # cached weights (Section 5 inference pipeline) give the same y
    out2 = quest.quest_linear_fwd(x, None, bits, g, trust, out_dtype=out_dtype,
                                  w_cached={"wq": out["wq"], "sw": out["sw"]})
    torch.cuda.synchronize()
    assert torch.equal(out2["y"], out["y"]) and torch.equal(out2["xq"], out["xq"])
    return out


def test_config1():
    c = synth.config1()
    check_linear(c["x"], c["w"], 4, 512, 1.0, torch.float32, F32_IN_RTOL)


@pytest.mark.parametrize("g", [128, 2048])
def test_config2(g):
    c = synth.config2()
    rows = np.random.default_rng(0).choice(4096, 128, replace=False)
    check_linear(c["x"], c["w"], 4, g, 1.0, torch.bfloat16, BF16_OUT_RTOL, sample_rows=rows)


@pytest.mark.parametrize("bits,trust", [(1, 1.0), (1, 1.3), (2, 1.0)])
def test_config3(bits, trust):
    c = synth.config2()
    rows = np.random.default_rng(1).choice(4096, 128, replace=False)
    check_linear(c["x"], c["w"], bits, 128, trust, torch.bfloat16, BF16_OUT_RTOL, sample_rows=rows)


def test_config4_layers_one_call_each():
    """The three layers of config 4 as separate quest_linear_fwd calls with the SwiGLU as torch glue (the
    fused block is tested in test_gpu_mlp.py); the oracle for the down projection is fed the GPU's own
    bf16 hidden activations."""
    import paper_2502_05003_b200 as quest
    c = synth.config4()
    rows = np.random.default_rng(2).choice(8192, 64, replace=False)
    gate = check_linear(c["x"], c["w_gate"], 4, 128, 1.0, torch.bfloat16, BF16_OUT_RTOL, sample_rows=rows)["y"]
    up = quest.quest_linear_fwd(to_dev(c["x"]), to_dev(c["w_up"]), 4, 128, out_dtype=torch.bfloat16)["y"]
    h = (torch.nn.functional.silu(gate.float()) * up.float()).to(torch.bfloat16)
    h_np = h.view(torch.int16).cpu().numpy().view(np.uint16)
    check_linear(h_np, c["w_down"], 4, 128, 1.0, torch.bfloat16, BF16_OUT_RTOL, sample_rows=rows)


@pytest.mark.parametrize("bits", [1, 2, 3, 4, 8])
@pytest.mark.parametrize("d,tokens", [(512, 1024), (1024, 1024), (4096, 1024), (2048, 16384)])
def test_config5_points(bits, d, tokens):
    p = synth.config5_point(bits * 10 + d // 512, tokens, d)
    rows = np.random.default_rng(3).choice(tokens, 32, replace=False)
    for g in (128, d):
        check_linear(p["x"], p["w"], bits, g, 1.0, torch.bfloat16, BF16_OUT_RTOL, sample_rows=rows)


def test_large_layer_quantized_by_the_block_kernel():
    """x and w of 32 Mi elements together: the quantizer launch with one thread per rotation block writes codes,
    masks and the tensor-core operands of both tensors (8-bit codes stay on the kernels that also sum the rows)."""
    p = synth.config5_point(7, 16384, 2048)
    rows = np.random.default_rng(5).choice(16384, 24, replace=False)
    check_linear(p["x"], p["w"], 4, 128, 1.0, torch.bfloat16, BF16_OUT_RTOL, sample_rows=rows)
    check_linear(p["x"], p["w"], 2, 128, 1.0, torch.bfloat16, BF16_OUT_RTOL, sample_rows=rows)
    check_linear(p["x"], p["w"], 8, 128, 1.0, torch.bfloat16, BF16_OUT_RTOL, sample_rows=rows)


def test_linear_fwd_in_two_calls_equals_the_single_call():
    """quest_linear_fwd_quantize followed by quest_linear_fwd_contract is quest_linear_fwd, bit for bit."""
    import paper_2502_05003_b200 as quest
    for bits, M, N, K in ((4, 300, 200, 512), (8, 136, 264, 256), (2, 257, 130, 384)):
        p = synth.config5_point(bits, M, K)
        x, w = to_dev(p["x"]), to_dev(synth.f32_to_bf16_bits(synth.weights(N, K, np.random.default_rng(bits))))
        ref = quest.quest_linear_fwd(x, w, bits, 128, 1.0, out_dtype=torch.bfloat16)
        saved = {k: torch.zeros_like(ref[k]) for k in ("xq", "sx", "mx", "wq", "sw", "mw")}
        ws = quest.alloc_workspace(M, N, K, bits, bits)
        y = torch.zeros_like(ref["y"])
        quest.quest_linear_fwd_quantize(x, w, bits, 128, 1.0, saved, ws)
        quest.quest_linear_fwd_contract(saved, M, N, K, bits, y, ws)
        torch.cuda.synchronize()
        for k in saved:
            assert torch.equal(saved[k], ref[k]), k
        assert torch.equal(y, ref["y"])
        # the second half alone can be repeated: the operands stay in the workspace
        y.zero_()
        quest.quest_linear_fwd_contract(saved, M, N, K, bits, y, ws)
        torch.cuda.synchronize()
        assert torch.equal(y, ref["y"])


def test_linear_fwd_replays_from_a_cuda_graph():
    """Section 5 runs the whole pipeline under a CUDA graph: the call must be capturable (no
    allocation, no synchronisation) and every replay must reproduce the directly launched result."""
    import paper_2502_05003_b200 as quest
    c = synth.config2(tokens=512)
    x, w = to_dev(c["x"]), to_dev(c["w"])
    ref = quest.quest_linear_fwd(x, w, 4, 128, 1.0, out_dtype=torch.bfloat16)
    M, K = x.shape
    N = w.shape[0]
    saved = {"xq": torch.zeros_like(ref["xq"]), "sx": torch.zeros_like(ref["sx"]), "mx": torch.zeros_like(ref["mx"]),
             "wq": torch.zeros_like(ref["wq"]), "sw": torch.zeros_like(ref["sw"]), "mw": torch.zeros_like(ref["mw"])}
    y = torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")
    ws = quest.alloc_workspace(M, N, K, 4, 4)
    torch.cuda.synchronize()
    st = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(st):
        quest.quest_linear_fwd(x, w, 4, 128, 1.0, y=y, saved=saved, workspace=ws)     # warm-up outside the capture
        st.synchronize()
        with torch.cuda.graph(g, stream=st):
            quest.quest_linear_fwd(x, w, 4, 128, 1.0, y=y, saved=saved, workspace=ws)
    for _ in range(3):
        y.zero_()
        for t in saved.values():
            t.zero_()
        g.replay()
        torch.cuda.synchronize()
        assert torch.equal(y, ref["y"])
        for k in saved:
            assert torch.equal(saved[k], ref[k]), k
    assert quest.quest_device_status() == 0


def test_two_streams_share_no_hidden_state():
    """Calls on different streams with their own workspaces may overlap on the GPU: the library keeps
    no mutable state between calls (apart from the timeout word), so both results equal the serial ones."""
    import paper_2502_05003_b200 as quest
    rng = np.random.default_rng(11)
    xs = [to_dev(synth.f32_to_bf16_bits(rng.standard_normal((1024, 1024)).astype(np.float32))) for _ in range(2)]
    ws = [to_dev(synth.f32_to_bf16_bits((rng.standard_normal((768, 1024)) * 0.02).astype(np.float32))) for _ in range(2)]
    serial = [quest.quest_linear_fwd(xs[i], ws[i], 4, 128, 1.0, out_dtype=torch.bfloat16) for i in range(2)]
    torch.cuda.synchronize()
    streams = [torch.cuda.Stream() for _ in range(2)]
    outs = [None, None]
    for rep in range(5):
        for i in range(2):
            with torch.cuda.stream(streams[i]):
                outs[i] = quest.quest_linear_fwd(xs[i], ws[i], 4, 128, 1.0, out_dtype=torch.bfloat16)
        torch.cuda.synchronize()
        for i in range(2):
            for k in ("y", "xq", "mx", "wq", "mw", "sx", "sw"):
                assert torch.equal(outs[i][k], serial[i][k]), (rep, i, k)
    assert quest.quest_device_status() == 0


@pytest.mark.parametrize("bits", [2, 4, 8])
def test_cached_weight_operand_is_reused_across_calls_with_other_row_counts(bits):
    """w_is_cached = 2: the operand of w left in the workspace by an earlier call serves later calls."""
    import paper_2502_05003_b200 as quest
    rng = np.random.default_rng(40 + bits)
    N, K, g = 264, 512, 128
    w = torch.from_numpy(synth.f32_to_bf16_bits((rng.standard_normal((N, K)) * 0.02).astype(np.float32))).view(torch.bfloat16).cuda()
    xs = [torch.from_numpy(synth.f32_to_bf16_bits(rng.standard_normal((M, K)).astype(np.float32))).view(torch.bfloat16).cuda()
          for M in (300, 130, 520)]
    ws = quest.alloc_workspace(520, N, K, bits, bits)
    first = quest.quest_linear_fwd(xs[0], w, bits, g, workspace=ws)
    cached = {"wq": first["wq"], "sw": first["sw"], "operand_in_workspace": True}
    for x in xs[1:]:
        got = quest.quest_linear_fwd(x, None, bits, g, w_cached=cached, workspace=ws)
        ref = quest.quest_linear_fwd(x, w, bits, g)
        torch.cuda.synchronize()
        assert torch.equal(got["y"], ref["y"]) and torch.equal(got["xq"], ref["xq"])
    assert quest.quest_device_status() == 0
