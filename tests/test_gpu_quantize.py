"""GPU parity: quest_quantize / quest_trust_mask through the C ABI against the CPU oracle.
Codes and masks bit-exact; scales within 1e-5 relative."""
import numpy as np
import pytest
import torch

from oracle import quest_oracle as qo
from paper_2502_05003_b200 import synth
from tests.gpu_util import canary_intact, guarded, to_dev

pytestmark = pytest.mark.gpu

SCALE_RTOL = 1e-5


def check(x_np, bits, g, trust=1.0, repeat=2):
    import paper_2502_05003_b200 as quest
    ref = qo.quantize(x_np, bits, g, trust)
    x = to_dev(x_np)
    rows, cols = x_np.shape
    cb = quest.container_bits(bits)
    for _ in range(repeat):
        raw_c, codes, n_c = guarded((rows, cols * cb // 8), torch.uint8)
        raw_m, mask, n_m = guarded((rows, cols // 8), torch.uint8)
        raw_s, scales, n_s = guarded((rows,), torch.float32)
        quest.quest_quantize(x, bits, g, trust, codes=codes, scales=scales, mask=mask)
        torch.cuda.synchronize()
        assert canary_intact(raw_c, n_c) and canary_intact(raw_m, n_m) and canary_intact(raw_s, n_s)
        c, m, s = codes.cpu().numpy(), mask.cpu().numpy(), scales.cpu().numpy()
        assert np.array_equal(c, ref["codes"]), f"codes differ in {(c != ref['codes']).sum()} bytes"
        assert np.array_equal(m, ref["mask"]), f"mask differs in {(m != ref['mask']).sum()} bytes"
        assert np.allclose(s, ref["scales"], rtol=SCALE_RTOL, atol=0)
    m2 = quest.quest_trust_mask(x, bits, g, trust)
    torch.cuda.synchronize()
    assert np.array_equal(m2.cpu().numpy(), ref["mask"])
    assert quest.quest_device_status() == 0


def rows_of(kind, rows, cols, seed, bf16):
    rng = np.random.default_rng(seed)
    if kind == "gauss":
        a = rng.standard_normal((rows, cols)).astype(np.float32)
    elif kind == "outliers":
        a = synth.gaussian_with_outliers(rows, cols, rng)
    elif kind == "student":
        a = synth.student_t(rows, cols, rng)
    elif kind == "channels":
        a = synth.channel_scaled_gaussian(rows, cols, rng)
    elif kind == "small":
        a = synth.weights(rows, cols, rng)
    return synth.f32_to_bf16_bits(a) if bf16 else a


@pytest.mark.parametrize("bits", [1, 2, 3, 4, 5, 8])
@pytest.mark.parametrize("g,cols", [(1, 64), (8, 256), (32, 96), (64, 640), (128, 128), (128, 2048), (128, 5504),
                                    (256, 768), (512, 512), (1024, 1024), (1024, 3072), (2048, 2048), (2048, 4096),
                                    (4096, 4096)])
def test_bf16_rows(bits, g, cols):
    check(rows_of("student", 67, cols, bits * 100 + g, True), bits, g)


@pytest.mark.parametrize("bits", [1, 2, 3, 4, 8])
@pytest.mark.parametrize("dtype_bf16", [False, True])
@pytest.mark.parametrize("g,cols", [(8, 8), (8, 24), (1, 40), (8, 72), (8, 136), (4, 1000), (8, 4104), (2, 16376)])
def test_row_lengths_that_are_not_multiples_of_32(bits, dtype_bf16, g, cols):
    check(rows_of("outliers", 19, cols, bits + cols, dtype_bf16), bits, g)


@pytest.mark.parametrize("bits", [1, 4, 8])
@pytest.mark.parametrize("g,cols", [(16, 48), (128, 1280), (512, 512), (2048, 2048), (8192, 8192), (16384, 16384)])
def test_f32_rows(bits, g, cols):
    check(rows_of("outliers", 33, cols, bits * 7 + g, False), bits, g)


@pytest.mark.parametrize("trust", [0.5, 1.0])
@pytest.mark.parametrize("bits", [1, 4, 8])
@pytest.mark.parametrize("g,cols", [(128, 16384), (64, 8256), (4096, 16384), (16384, 16384), (8192, 8192), (128, 8320),
                                    (256, 12288)])
def test_bf16_rows_wider_than_8192(g, cols, bits, trust):
    """Rows of more than 8192 bfloat16 elements take the persistent streaming kernel (64 elements per
    thread): its specialised tail (g = 128, trust_factor >= 1) and its general one, with the first
    butterfly stage read from shared memory (g >= 128) or from registers (g = 64), and rotation blocks
    that span several warps (g >= 4096).  (8192, 8192) is the widest block the 32-per-thread kernel
    serves through its shared-memory exchange."""
    check(rows_of("student", 37, cols, bits * 31 + g + cols, True), bits, g, trust)


@pytest.mark.parametrize("cols,bits,trust", [(2048, 4, 1.0), (2048, 1, 1.3), (2048, 2, 1.0), (2048, 8, 1.0), (128, 4, 1.0),
                                             (256, 3, 1.0), (1024, 4, 2.0), (4096, 4, 1.0), (640, 4, 1.0), (5504, 4, 1.0),
                                             (5504, 8, 1.0), (8320, 2, 1.0), (16384, 4, 1.0), (12288, 1, 1.0)])
def test_large_tensors_one_thread_per_rotation_block(cols, bits, trust):
    """From 32 Mi elements on, dense bfloat16 tensors with had_block = 128 and trust_factor >= 1 take the kernel in
    which one thread owns a whole rotation block: rows whose blocks fill part of a warp (cols = 128 .. 4096, block
    sums combined by shuffles) and rows that span warps or have a number of blocks that is not a power of two
    (through shared memory), with a ragged last CTA in every case."""
    rows = (32 << 20) // cols + 37
    check(rows_of("gauss", rows, cols, cols + bits, True), bits, 128, trust, repeat=1)


@pytest.mark.parametrize("trust", [0.0, 0.5, 1.0, 1.25, 1.3, 3.0])
@pytest.mark.parametrize("bits", [1, 2, 4])
def test_trust_factors(bits, trust):
    check(rows_of("gauss", 64, 1024, 5, True), bits, 128, trust)


def test_edge_rows():
    import paper_2502_05003_b200 as quest
    cols = 512
    x = np.zeros((9, cols), np.float32)
    x[1, :] = 2.5                       # constant row
    x[2, 100] = 1e6                     # single spike
    x[3, :] = np.where(np.arange(cols) % 2 == 0, 1.0, -1.0)   # one Hadamard basis vector
    x[4, :] = 1e-30                     # tiny values (subnormal squares)
    x[5, :] = 1e18                      # huge values
    x[6, :] = np.linspace(-1, 1, cols)
    x[7, ::7] = -3.0
    x[8, :] = np.arange(cols) - 255.5   # exact half-integers: rounding ties
    for bits in (1, 2, 4, 8):
        for g in (1, 128, 512):
            check(x, bits, g)
            check(synth.f32_to_bf16_bits(x), bits, g)
    # empty input is a no-op
    e = torch.empty((0, 128), dtype=torch.float32, device="cuda")
    c, s, m = quest.quest_quantize(e, 4, 128)
    assert c.shape == (0, 64) and s.shape == (0,)


def test_strided_rows():
    import paper_2502_05003_b200 as quest
    x_np = rows_of("student", 40, 1024, 3, True)
    big = to_dev(np.concatenate([x_np, x_np], axis=1))           # ld = 2048
    view = big[:, :1024]
    codes, scales, mask = quest.quest_quantize(view, 4, 128)
    ref = qo.quantize(x_np, 4, 128)
    assert np.array_equal(codes.cpu().numpy(), ref["codes"]) and np.array_equal(mask.cpu().numpy(), ref["mask"])


def test_config1_full():
    c = synth.config1()
    check(c["x"], 4, 512)
    check(c["w"], 4, 512)


@pytest.mark.parametrize("g", [128, 2048])
@pytest.mark.parametrize("bits,trust", [(4, 1.0), (1, 1.0), (1, 1.3), (2, 1.0)])
def test_config2_and_3_full_size(g, bits, trust):
    c = synth.config2()
    check(c["x"], bits, g, trust, repeat=1)
    check(c["w"], bits, g, trust, repeat=1)


def test_config4_inputs_full_size():
    c = synth.config4()
    check(c["x"], 4, 128, repeat=1)
    check(c["w_gate"], 4, 128, repeat=1)
    check(c["w_down"], 4, 128, repeat=1)          # K = 5504 = 43 blocks of 128
    rng = np.random.default_rng(9)
    h = synth.f32_to_bf16_bits(rng.standard_normal((8192, 5504)).astype(np.float32) ** 2)
    check(h, 4, 128, repeat=1)


def test_argument_errors_raise():
    import paper_2502_05003_b200 as quest
    x = torch.zeros((4, 128), dtype=torch.float32, device="cuda")
    for kw in (dict(bits=0, had_block=128), dict(bits=4, had_block=48), dict(bits=4, had_block=128, trust_factor=-1)):
        with pytest.raises(quest.QuestError):
            quest.quest_quantize(x, **kw)
    with pytest.raises(ValueError):
        quest.quest_quantize(x.cpu(), 4, 128)
