"""GPU parity for the FP4 (E2M1) grid variant through the C ABI: codes, masks and the int32
accumulators (four times the value product) bit-exact with the oracle; scales within 1e-5; outputs
within the tolerances of the uniform-grid tests."""
import numpy as np
import pytest
import torch

from oracle import quest_oracle as qo
from paper_2502_05003_b200 import synth
from tests.gpu_util import assert_output_close, to_dev

pytestmark = pytest.mark.gpu


def check_quantize(x_np, g, trust=1.0):
    import paper_2502_05003_b200 as quest
    ref = qo.quantize_fp4(x_np, g, trust)
    codes, scales, mask = quest.quest_quantize_fp4(to_dev(x_np), g, trust)
    torch.cuda.synchronize()
    c, m = codes.cpu().numpy(), mask.cpu().numpy()
    assert np.array_equal(c, ref["codes"]), f"codes differ in {(c != ref['codes']).sum()} bytes"
    assert np.array_equal(m, ref["mask"]), f"mask differs in {(m != ref['mask']).sum()} bytes"
    assert np.allclose(scales.cpu().numpy(), ref["scales"], rtol=1e-5, atol=0)
    return ref


def rows(kind, r, c, seed, bf16=True):
    rng = np.random.default_rng(seed)
    a = {"gauss": lambda: rng.standard_normal((r, c)).astype(np.float32),
         "student": lambda: synth.student_t(r, c, rng),
         "outliers": lambda: synth.gaussian_with_outliers(r, c, rng)}[kind]()
    return synth.f32_to_bf16_bits(a) if bf16 else a


@pytest.mark.parametrize("g,cols", [(1, 64), (32, 96), (128, 128), (128, 2048), (128, 5504), (512, 512), (2048, 2048),
                                    (4096, 4096)])
@pytest.mark.parametrize("bf16", [True, False])
def test_quantize_shapes(g, cols, bf16):
    check_quantize(rows("student", 67, cols, g + cols, bf16), g)


@pytest.mark.parametrize("trust", [0.5, 1.0])
@pytest.mark.parametrize("g,cols", [(128, 16384), (64, 8256), (4096, 16384), (16384, 16384), (8192, 8192)])
def test_quantize_bf16_rows_wider_than_8192(g, cols, trust):
    """The persistent streaming kernel (rows of more than 8192 bfloat16 elements) with the FP4 grid:
    specialised and general tails."""
    check_quantize(rows("student", 37, cols, g + cols + 1), g, trust)


@pytest.mark.parametrize("cols", [2048, 5504])
def test_quantize_large_tensors_one_thread_per_rotation_block(cols):
    """The kernel that serves dense bfloat16 tensors of 32 Mi elements and more, with the FP4 grid."""
    check_quantize(rows("gauss", (32 << 20) // cols + 37, cols, cols), 128, 1.0)


@pytest.mark.parametrize("trust", [0.0, 0.5, 1.0, 1.3, 3.0])
def test_trust_factors(trust):
    check_quantize(rows("gauss", 64, 1024, 5), 128, trust)


def test_edge_rows_and_hardware_rounding_on_exact_ties():
    cols = 512
    x = np.zeros((6, cols), np.float32)
    x[1, :] = 2.5
    x[2, 100] = 1e6
    x[3, :] = np.where(np.arange(cols) % 2 == 0, 1.0, -1.0)
    x[4, :] = np.linspace(-1, 1, cols)
    x[5, :] = np.tile(np.array([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0, 6.0], np.float32), cols // 8) * \
        np.where(np.arange(cols) % 16 < 8, 1.0, -1.0)
    for g in (1, 128):
        check_quantize(x, g)
        check_quantize(synth.f32_to_bf16_bits(x), g)


def test_config2_full_size():
    c = synth.config2()
    check_quantize(c["x"], 128)
    check_quantize(c["w"], 128)


@pytest.mark.parametrize("M,N,K", [(128, 128, 128), (37, 29, 96), (300, 1000, 2048), (513, 136, 5504)])
def test_gemm_accumulators_bit_exact(M, N, K):
    import paper_2502_05003_b200 as quest
    rng = np.random.default_rng(M + N + K)
    xq = rng.integers(0, 256, size=(M, K // 2), dtype=np.uint8)
    wq = rng.integers(0, 256, size=(N, K // 2), dtype=np.uint8)
    sx = (rng.random(M) + 0.5).astype(np.float32)
    sw = (rng.random(N) * 0.01 + 0.001).astype(np.float32)
    d = lambda a: torch.from_numpy(a).cuda()
    y, acc = quest.quest_lowbit_gemm_fp4(d(xq), d(sx), d(wq), d(sw), K, out_dtype=torch.float32, want_acc=True)
    torch.cuda.synchronize()
    ref_acc = qo.gemm_acc_fp4(xq, wq, K)
    assert np.array_equal(acc.cpu().numpy(), ref_acc)
    ref_y = qo.dequant_fp4(ref_acc, sx, sw)
    got = y.cpu().numpy().astype(np.float64)
    assert np.all(np.abs(got - ref_y) <= 1e-5 * np.abs(ref_y) + 1e-30)
    assert quest.quest_device_status() == 0


def test_gemm_accumulators_exact_at_the_largest_sum():
    # every product is +36 (6 x 6) or -36 over the longest supported row: |acc4| = 4 * 36 * K = 9.4 M < 2^24,
    # the largest value the binary32 accumulators of the FP4 tensor-core path must hold exactly
    import paper_2502_05003_b200 as quest
    M, N, K = 130, 136, 65504
    xq = np.full((M, K // 2), 0x77, np.uint8)               # +6, +6
    xq[1::2] = 0xF7                                          # rows alternate: (+6, -6) pairs cancel
    xq[2::3, : K // 4] = 0xFF                                # and some rows start with -6
    wq = np.full((N, K // 2), 0x77, np.uint8)
    wq[::5] = 0xFF
    ones_m, ones_n = np.ones(M, np.float32), np.ones(N, np.float32)
    d = lambda a: torch.from_numpy(a).cuda()
    y, acc = quest.quest_lowbit_gemm_fp4(d(xq), d(ones_m), d(wq), d(ones_n), K, out_dtype=torch.float32, want_acc=True)
    torch.cuda.synchronize()
    ref = qo.gemm_acc_fp4(xq, wq, K)
    assert np.abs(ref).max() == 4 * 36 * K
    assert np.array_equal(acc.cpu().numpy(), ref)
    assert np.array_equal(y.cpu().numpy().astype(np.float64) * 4.0, ref.astype(np.float64))
    assert quest.quest_device_status() == 0


@pytest.mark.parametrize("g", [128, 2048])
def test_linear_fwd_config2(g):
    import paper_2502_05003_b200 as quest
    c = synth.config2()
    out = quest.quest_linear_fwd_fp4(to_dev(c["x"]), to_dev(c["w"]), g, 1.0, out_dtype=torch.bfloat16)
    torch.cuda.synchronize()
    qx, qw = qo.quantize_fp4(c["x"], g), qo.quantize_fp4(c["w"], g)
    for k, ref in (("xq", qx["codes"]), ("mx", qx["mask"]), ("wq", qw["codes"]), ("mw", qw["mask"])):
        assert np.array_equal(out[k].cpu().numpy(), ref), k
    rows_ = np.sort(np.random.default_rng(0).choice(4096, 96, replace=False))
    ref_y = qo.dequant_fp4(qo.gemm_acc_fp4(qx["codes"][rows_], qw["codes"], 2048), qx["scales"][rows_], qw["scales"])
    got = out["y"].float().cpu().numpy().astype(np.float64)[rows_]
    assert_output_close(got, ref_y, True)
    # cached weights give the same result
    out2 = quest.quest_linear_fwd_fp4(to_dev(c["x"]), None, g, 1.0, out_dtype=torch.bfloat16,
                                      w_cached={"wq": out["wq"], "sw": out["sw"]})
    torch.cuda.synchronize()
    assert torch.equal(out2["y"], out["y"])
    # sanity: the quantized product approximates x w^T about as well as a 4-bit format can
    x64 = synth.bf16_bits_to_f32(c["x"][rows_]).astype(np.float64)
    w64 = synth.bf16_bits_to_f32(c["w"]).astype(np.float64)
    exact = x64 @ w64.T
    assert np.linalg.norm(got - exact) / np.linalg.norm(exact) < 0.25
