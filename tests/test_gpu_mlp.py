"""GPU parity: quest_mlp_fwd (gate / up / SwiGLU / down, every linear layer Algorithm 1) through the C ABI.

Against ``oracle/mlp.py``: codes, masks and scales of x, w_gate, w_up bit-exact (scales to 1e-5); the hidden
activations h within the rounding of their bfloat16 storage (gate, up and silu are evaluated in binary32 on the
GPU and in binary64 by the oracle: about 1e-6 relative, far inside the 2^-8 of the format); then the down
projection with the oracle fed the GPU's own stored h, so that its codes, masks and scales are bit-exact again
and y is within the output tolerance.
"""
import numpy as np
import pytest
import torch

from oracle import mlp as om
from paper_2502_05003_b200 import synth
from tests.gpu_util import assert_output_close, to_dev

pytestmark = pytest.mark.gpu


def bits_of(t: torch.Tensor) -> np.ndarray:
    return t.view(torch.int16).cpu().numpy().view(np.uint16)


def check_block(x, wg, wu, wd, bits, g, trust=1.0, rows=None, out_dtype=torch.bfloat16):
    import paper_2502_05003_b200 as quest
    out = quest.quest_mlp_fwd(to_dev(x), to_dev(wg), to_dev(wu), to_dev(wd), bits, g, trust, out_dtype=out_dtype)
    torch.cuda.synchronize()
    assert quest.quest_device_status() == 0
    ref = om.hidden(x, wg, wu, bits, g, trust, rows=rows)
    for name, q in (("x", ref["x"]), ("wg", ref["w_gate"]), ("wu", ref["w_up"])):
        c, s, m = {"x": ("xq", "sx", "mx"), "wg": ("wgq", "swg", "mwg"), "wu": ("wuq", "swu", "mwu")}[name]
        assert np.array_equal(out[c].cpu().numpy(), q["codes"]), f"{name}: codes"
        assert np.array_equal(out[m].cpu().numpy(), q["mask"]), f"{name}: mask"
        assert np.allclose(out[s].cpu().numpy(), q["scales"], rtol=1e-5, atol=0), f"{name}: scales"
    r = ref["rows"]
    h_bits = bits_of(out["h"])
    got_h = synth.bf16_bits_to_f32(h_bits[r]).astype(np.float64)
    assert_output_close(got_h, ref["h"], True)
    # down projection on the stored hidden activations
    d = om.down_from_hidden(h_bits, wd, bits, g, trust, rows=rows)
    assert np.array_equal(out["hq"].cpu().numpy(), d["h"]["codes"]), "h: codes"
    assert np.array_equal(out["mh"].cpu().numpy(), d["h"]["mask"]), "h: mask"
    assert np.allclose(out["sh"].cpu().numpy(), d["h"]["scales"], rtol=1e-5, atol=0)
    assert np.array_equal(out["wdq"].cpu().numpy(), d["w_down"]["codes"]) and np.array_equal(out["mwd"].cpu().numpy(), d["w_down"]["mask"])
    assert np.allclose(out["swd"].cpu().numpy(), d["w_down"]["scales"], rtol=1e-5, atol=0)
    got_y = out["y"].float().cpu().numpy().astype(np.float64)[r]
    assert_output_close(got_y, d["y"], out_dtype == torch.bfloat16)
    return out


def block_inputs(T, H, I, seed, bf16=True):
    rng = np.random.default_rng(seed)
    c = (lambda a: synth.f32_to_bf16_bits(a)) if bf16 else (lambda a: a)
    return (c(synth.student_t(T, H, rng)), c(synth.weights(I, H, rng)), c(synth.weights(I, H, rng)),
            c(synth.weights(H, I, rng)))


@pytest.mark.parametrize("T,H,I,g", [(300, 256, 384, 128), (64, 128, 128, 128), (136, 512, 640, 128), (520, 256, 192, 64),
                                     (8, 64, 96, 32), (257, 384, 1000 // 8 * 8 + 24, 8)])
def test_shapes(T, H, I, g):
    check_block(*block_inputs(T, H, I, T + H + I), 4, g)


@pytest.mark.parametrize("bits", [1, 2, 3, 5, 8])
def test_bit_widths(bits):
    check_block(*block_inputs(264, 256, 384, bits), bits, 128)


def test_trust_factor_and_binary32_inputs_and_outputs():
    check_block(*block_inputs(200, 256, 256, 3), 1, 128, trust=1.3)
    check_block(*block_inputs(200, 256, 256, 4, bf16=False), 4, 128, out_dtype=torch.float32)


def test_config4_mlp_block():
    """Config 4 at full size (X[8192 x 2048], MLP width 5504) on sampled token rows."""
    c = synth.config4()
    rows = np.random.default_rng(2).choice(8192, 48, replace=False)
    check_block(c["x"], c["w_gate"], c["w_up"], c["w_down"], 4, 128, rows=rows)


def test_replay_from_a_cuda_graph_and_preallocated_buffers():
    import paper_2502_05003_b200 as quest
    x, wg, wu, wd = [to_dev(a) for a in block_inputs(512, 256, 384, 9)]
    ref = quest.quest_mlp_fwd(x, wg, wu, wd, 4, 128)
    bufs = quest.mlp_buffers(512, 256, 384, 4)
    for k, v in bufs.items():
        if torch.is_tensor(v):
            v.zero_()
    st = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(st):
        quest.quest_mlp_fwd(x, wg, wu, wd, 4, 128, buffers=bufs)
        st.synchronize()
        with torch.cuda.graph(g, stream=st):
            quest.quest_mlp_fwd(x, wg, wu, wd, 4, 128, buffers=bufs)
    for k in ("h", "y", "hq"):
        bufs[k].zero_()
    g.replay()
    torch.cuda.synchronize()
    for k in ("h", "y", "xq", "hq", "mh", "sh", "wdq"):
        assert torch.equal(bufs[k], ref[k]), k
    assert quest.quest_device_status() == 0


def test_argument_errors():
    import paper_2502_05003_b200 as quest
    x, wg, wu, wd = [to_dev(a) for a in block_inputs(64, 128, 128, 1)]
    with pytest.raises(quest.QuestError):
        quest.quest_mlp_fwd(x, wg, wu, wd, 0, 128)
    with pytest.raises(quest.QuestError):
        quest.quest_mlp_fwd(x, wg, wu, wd, 4, 96)
    with pytest.raises(ValueError):
        quest.quest_mlp_fwd(x, wg, wu[:, :64].contiguous(), wd, 4, 128)
