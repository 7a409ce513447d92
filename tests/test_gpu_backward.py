"""GPU parity: quest_linear_bwd (Algorithm 2) through the C ABI against the binary64 oracle.

What the CUDA path rounds: one operand of every product is dequantised to bfloat16 (relative error at
most u = 2^-8, the unit roundoff of an 8-bit significand; the other operand, dy, is bfloat16 already,
and the products are exact in binary32), and the sum over the contraction index runs in binary32 on the
tensor cores (N additions, each within 2^-24 of the running sum).  So the masked product-sum d[i][k]
is off by at most  (u + N 2^-24) * T1[i][k],  T1[i][k] = sum_n |dy[i][n] q[n][k]|.  The inverse Hadamard
transform adds, per output element, the errors of its block with weights +-g^-1/2 (in binary32:
log2 g more roundings), so

    |got[i][j] - ref[i][j]| <= (u + (N + 8 log2 g) 2^-24) * g^-1/2 * sum_{k in block(j)} T1[i][k]     (hard)

element by element, plus u |ref| when the output is stored as bfloat16.  That bound is rigorous but
loose, because rounding errors do not all point the same way: a single wrongly applied mask bit moves
an output by g^-1/2 |d[i][k]|, about (sum_n t_n^2)^(1/2), which can hide under it once N is large.
So a second, statistical bound is asserted per row and rotation block: independent rounding errors of
relative size up to u have standard deviation u/sqrt(3) times the term, hence the error vector of one
block (128 or g numbers; the transform is orthonormal) has a Euclidean norm close to

    (u / sqrt(3)) * ( sum_{k in block} T2[i][k] )^(1/2),   T2[i][k] = sum_n (dy[i][n] q[n][k])^2,

and the test allows four times that (a g-element norm concentrates well inside 4x; for g < 32 the
block is padded with its neighbours up to 32 elements).  A wrong mask bit adds the whole of
d[i][k]^2, roughly T2[i][k], to the squared norm: thousands of times the allowance.
"""
import numpy as np
import pytest
import torch

from oracle import backward as ob
from oracle import quest_oracle as qo
from paper_2502_05003_b200 import synth
from tests.gpu_util import to_dev

pytestmark = pytest.mark.gpu

U_BF16 = 2.0 ** -8


def run_case(x_np, w_np, bits, g, seed=0, out_dtype=torch.float32, rows_x=None, rows_w=None, edit_masks=None):
    import paper_2502_05003_b200 as quest
    M, K = x_np.shape
    N = w_np.shape[0]
    fx, fw = qo.quantize(x_np, bits, g), qo.quantize(w_np, bits, g)
    if edit_masks is not None:                  # any bitmap is a valid input of Algorithm 2
        edit_masks(fx["mask"], fw["mask"])
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
    xh = fx["scales"].astype(np.float64)[:, None] * ob.grid_values(fx["codes"], K, bits)
    wh = fw["scales"].astype(np.float64)[:, None] * ob.grid_values(fw["codes"], K, bits)
    mbx, mbw = ob.mask_bits(fx["mask"], K)[rx], ob.mask_bits(fw["mask"], K)[rw]
    # T1 = sum |terms|, T2 = sum terms^2 of every masked product-sum (zero where the mask drops it)
    t1x, t2x = mbx * (np.abs(dy64[rx]) @ np.abs(wh)), mbx * ((dy64[rx] ** 2) @ (wh ** 2))
    t1w, t2w = mbw * (np.abs(dy64[:, rw]).T @ np.abs(xh)), mbw * ((dy64[:, rw] ** 2).T @ (xh ** 2))
    store_u = U_BF16 if out_dtype == torch.bfloat16 else 2.0 ** -24
    for name, got_t, want, t1, t2, rows, nsum in (("dx", out["dx"], ref["dx"], t1x, t2x, rx, N),
                                                  ("dw", out["dw"], ref["dw"], t1w, t2w, rw, M)):
        got = got_t.float().cpu().numpy().astype(np.float64)[rows]
        err = np.abs(got - want)
        nb = K // g
        # hard element-wise bound
        unit = U_BF16 + (nsum + 8 * np.log2(max(g, 2))) * 2.0 ** -24
        blk1 = t1.reshape(len(rows), nb, g).sum(axis=2) / np.sqrt(g)                # [rows, blocks]
        lim = unit * np.repeat(blk1, g, axis=1) + store_u * np.abs(want) + 1e-30
        worst = np.max(err / lim)
        assert worst <= 1.0, f"{name}: an element at {worst:.3f} of the hard bound"
        # statistical bound per row and group of at least 32 transformed elements
        grp = max(g, 32)
        if K % grp == 0:
            e2 = (err ** 2).reshape(len(rows), K // grp, grp).sum(axis=2)
            s2 = t2.reshape(len(rows), K // grp, grp).sum(axis=2)
            w2 = (want ** 2).reshape(len(rows), K // grp, grp).sum(axis=2)
            allow = 4.0 * (U_BF16 / np.sqrt(3.0)) * np.sqrt(s2) + 4.0 * (store_u / np.sqrt(3.0)) * np.sqrt(w2) \
                + 2.0 ** -22 * np.sqrt(nsum) * np.sqrt(s2) + 1e-30
            worst = np.max(np.sqrt(e2) / allow)
            assert worst <= 1.0, f"{name}: a block at {worst:.3f} of the statistical bound"
        if g == 1:
            # no rotation: a masked element is an exact zero
            dropped = (mbx if name == "dx" else mbw) == 0
            assert np.all(got[dropped] == 0.0), f"{name}: masked elements are not exact zeros"
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


def _drop_rows_and_blocks(mx, mw):
    """Extreme bitmaps: a row that trusts nothing, a fully masked rotation block of 128, an isolated
    masked element, and alternating bits."""
    for m in (mx, mw):
        m[3, :] = 0
        m[5, 16:32] = 0                       # elements 128..255 of row 5
        m[6, 0] &= 0xFE                       # element 0 of row 6
        m[7, :] = 0xAA
        m[m.shape[0] - 1, :] = 0              # the last row (ragged tile edge)


@pytest.mark.parametrize("M,N,K,g", [(264, 320, 1024, 128),     # products with the fused inverse transform
                                     (264, 320, 1024, 512),     # masked product stored, then the row transform kernel
                                     (72, 200, 512, 128),       # M below one tile: the unfused path for dL/dx
                                     (40, 48, 256, 1)])         # no rotation: masked elements are exact zeros
def test_extreme_masks(M, N, K, g):
    run_case(gauss(M, K, 21), gauss(N, K, 22, 0.02), 4, g, seed=K + g, edit_masks=_drop_rows_and_blocks)
    run_case(gauss(M, K, 21), gauss(N, K, 22, 0.02), 4, g, seed=K + g, edit_masks=_drop_rows_and_blocks,
             out_dtype=torch.bfloat16)


def test_config2_size_without_the_fused_transform():
    """The masked products at the benchmark size through the unfused path (g = 256: binary32 product,
    then the row transform kernel), on sampled rows."""
    c = synth.config2()
    rx = np.random.default_rng(3).choice(4096, 32, replace=False)
    rw = np.random.default_rng(4).choice(2048, 32, replace=False)
    run_case(c["x"], c["w"], 4, 256, seed=5, rows_x=rx, rows_w=rw)


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
