"""GPU parity: quest_lowbit_gemm through the C ABI against the oracle.  int32 accumulators
bit-exact; outputs within 1e-5 (fp32 out) / 2e-3 (bf16 out) relative."""
import numpy as np
import pytest
import torch

from oracle import quest_oracle as qo
from tests.gpu_util import assert_output_close, canary_intact, guarded
from tests.helpers import container_bits

pytestmark = pytest.mark.gpu


def random_codes(rows, K, bits, rng):
    cb = container_bits(bits)
    lev = rng.integers(0, 2 ** bits, size=(rows, K))
    per = 8 // cb
    out = np.zeros((rows, K // per), np.uint8)
    for e in range(per):
        out |= (lev[:, e::per].astype(np.uint8) << (e * cb)).astype(np.uint8)
    return out


def run_case(M, N, K, bx, bw, out_dtype, seed=0, sample_rows=None):
    import paper_2502_05003_b200 as quest
    rng = np.random.default_rng(seed)
    xq, wq = random_codes(M, K, bx, rng), random_codes(N, K, bw, rng)
    sx = (rng.random(M) + 0.5).astype(np.float32)
    sw = (rng.random(N) * 0.01 + 0.001).astype(np.float32)
    raw_y, y, n_y = guarded((M, N), out_dtype)
    raw_a, acc, n_a = guarded((M, N), torch.int32)
    d = lambda a: torch.from_numpy(a).cuda()
    quest.quest_lowbit_gemm(d(xq), d(sx), bx, d(wq), d(sw), bw, K, y=y, acc=acc)
    torch.cuda.synchronize()
    assert quest.quest_device_status() == 0
    assert canary_intact(raw_y, n_y) and canary_intact(raw_a, n_a)
    rows = np.arange(M) if sample_rows is None else np.asarray(sample_rows)
    ref_acc = qo.gemm_acc(xq[rows], bx, wq, bw, K)
    got_acc = acc.cpu().numpy()[rows]
    assert np.array_equal(got_acc, ref_acc), f"{(got_acc != ref_acc).sum()} accumulators differ"
    ref_y = qo.dequant(ref_acc, sx[rows], sw)
    got_y = y.float().cpu().numpy().astype(np.float64)[rows]
    assert_output_close(got_y, ref_y, out_dtype == torch.bfloat16)
    # y alone / acc alone
    y2, _ = quest.quest_lowbit_gemm(d(xq), d(sx), bx, d(wq), d(sw), bw, K, out_dtype=out_dtype)
    _, a2 = quest.quest_lowbit_gemm(d(xq), d(sx), bx, d(wq), d(sw), bw, K, want_y=False, want_acc=True)
    torch.cuda.synchronize()
    assert torch.equal(y2, y) and torch.equal(a2, acc)


@pytest.mark.parametrize("M,N,K", [(128, 128, 128), (128, 256, 256), (256, 512, 512), (1, 8, 32), (37, 29, 96),
                                   (130, 260, 160), (300, 1000, 2048), (513, 136, 5504), (64, 7, 64)])
@pytest.mark.parametrize("out_dtype", [torch.float32, torch.bfloat16])
def test_w4a4_shapes(M, N, K, out_dtype):
    run_case(M, N, K, 4, 4, out_dtype, seed=M + N + K)


@pytest.mark.parametrize("M,N,K", [(128, 128, 128), (1, 8, 32), (37, 29, 96), (130, 260, 160), (300, 1000, 2048),
                                   (513, 136, 5504), (64, 7, 64)])
@pytest.mark.parametrize("bits", [1, 2])
def test_one_and_two_bit_codes_on_the_fp4_path(M, N, K, bits):
    # both operands at most two bits wide: E2M1 nibble operands, kind::mxf4 contraction, exact integer sums
    run_case(M, N, K, bits, bits, torch.float32, seed=M + N + K + bits)


def test_two_bit_codes_at_the_longest_row_and_config3_size():
    import paper_2502_05003_b200 as quest
    K = 65504
    top = np.full((130, K // 4), 0xFF, np.uint8)        # every level 3 -> c = +3
    bot = np.zeros((136, K // 4), np.uint8)             # every level 0 -> c = -3
    ones = torch.ones(136, dtype=torch.float32, device="cuda")
    _, acc = quest.quest_lowbit_gemm(torch.from_numpy(top).cuda(), ones[:130], 2, torch.from_numpy(bot).cuda(), ones, 2,
                                     K, want_y=False, want_acc=True)
    assert bool((acc == -9 * K).all())
    rows = np.sort(np.random.default_rng(3).choice(4096, size=64, replace=False))
    run_case(4096, 2048, 2048, 1, 1, torch.bfloat16, seed=4, sample_rows=rows)
    run_case(4096, 2048, 2048, 2, 2, torch.bfloat16, seed=5, sample_rows=rows)


@pytest.mark.parametrize("bx,bw", [(1, 1), (2, 2), (1, 2), (2, 1), (2, 3), (3, 3), (8, 8), (4, 8), (8, 4), (1, 4), (5, 7)])
def test_bit_width_combinations(bx, bw):
    K = 1024 if max(bx, bw) < 8 else 512
    run_case(200, 328, K, bx, bw, torch.float32, seed=bx * 9 + bw)


def test_extreme_codes_do_not_overflow():
    import paper_2502_05003_b200 as quest
    K = 4096
    top = np.full((130, K // 2), 0xFF, np.uint8)        # every level 15 -> acc = K*225
    bot = np.zeros((140, K // 2), np.uint8)
    ones = torch.ones(140, dtype=torch.float32, device="cuda")
    _, acc = quest.quest_lowbit_gemm(torch.from_numpy(top).cuda(), ones[:130], 4, torch.from_numpy(bot).cuda(), ones, 4,
                                     K, want_y=False, want_acc=True)
    assert bool((acc == -K * 225).all())
    k8 = np.full((16, 33056), 255, np.uint8)
    with pytest.raises((quest.QuestError, ValueError)):  # K = 33056 at 8 bits could overflow int32: refused on the host
        quest.quest_lowbit_gemm(torch.from_numpy(k8).cuda(), ones[:16], 8, torch.from_numpy(k8).cuda(), ones[:16], 8,
                                33056)


def test_empty_product_is_a_no_op():
    import paper_2502_05003_b200 as quest
    xq = torch.empty((0, 64), dtype=torch.uint8, device="cuda")
    wq = torch.zeros((16, 64), dtype=torch.uint8, device="cuda")
    s = torch.ones(16, device="cuda")
    y, acc = quest.quest_lowbit_gemm(xq, s[:0], 4, wq, s, 4, 128, want_acc=True)
    assert y.shape == (0, 16) and acc.shape == (0, 16)


def test_config2_shape_sampled_rows():
    rows = np.random.default_rng(0).choice(4096, size=96, replace=False)
    run_case(4096, 2048, 2048, 4, 4, torch.bfloat16, seed=1, sample_rows=np.sort(rows))


def test_config4_down_projection_shape_sampled_rows():
    rows = np.random.default_rng(1).choice(8192, size=48, replace=False)
    run_case(8192, 2048, 5504, 4, 4, torch.bfloat16, seed=2, sample_rows=np.sort(rows))


def test_repeatable():
    import paper_2502_05003_b200 as quest
    rng = np.random.default_rng(5)
    xq = torch.from_numpy(random_codes(1024, 2048, 4, rng)).cuda()
    wq = torch.from_numpy(random_codes(768, 2048, 4, rng)).cuda()
    s1 = torch.rand(1024, device="cuda")
    s2 = torch.rand(768, device="cuda")
    outs = [quest.quest_lowbit_gemm(xq, s1, 4, wq, s2, 4, 2048, want_acc=True) for _ in range(3)]
    torch.cuda.synchronize()
    for y, a in outs[1:]:
        assert torch.equal(y, outs[0][0]) and torch.equal(a, outs[0][1])
