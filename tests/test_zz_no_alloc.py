"""quest_lowbit_gemm_static: the low-bit GEMM for callers that cannot allocate device memory.

Some users of this library only ever hold the pointers they are given: a plug-in inside a host
application, or a server whose own pools took all of device memory at start-up, so a later
cudaMalloc for a workspace fails.  For them the library keeps the GEMM's scratch in a fixed
array of its own.  These tests call that entry point through the C ABI with every output
preallocated and check it against the CPU oracle (int32 accumulators bit for bit, outputs within the
tolerance the other GEMM tests use) and against ``quest_lowbit_gemm``, which takes a caller-made
workspace.  The call is also watched for allocations: the free device memory the driver reports and
the bytes torch's allocator holds must both be the same after it as before.  Several calls run back to
back with different shapes and bit-widths, because the array is shared and keeps the previous
call's bytes.  The file sorts last so that a run stopping at the first failure has
already run every other test; it passes alone in a fresh process as well.
"""
import ctypes

import numpy as np
import pytest
import torch

from tests.helpers import container_bits


def _random_codes(rows, K, bits, rng):
    cb = container_bits(bits)
    lev = rng.integers(0, 2 ** bits, size=(rows, K))
    per = 8 // cb
    out = np.zeros((rows, K // per), np.uint8)
    for e in range(per):
        out |= (lev[:, e::per].astype(np.uint8) << (e * cb)).astype(np.uint8)
    return out


def _one_call(quest, M, N, K, bx, bw, out_dtype, seed):
    rng = np.random.default_rng(seed)
    d = lambda a: torch.from_numpy(a).cuda()
    xq, wq = d(_random_codes(M, K, bx, rng)), d(_random_codes(N, K, bw, rng))
    sx = d((rng.random(M) + 0.5).astype(np.float32))
    sw = d((rng.random(N) * 0.01 + 0.001).astype(np.float32))
    # reference: the existing entry point with a workspace the caller allocated
    y_ref, acc_ref = quest.quest_lowbit_gemm(xq, sx, bx, wq, sw, bw, K, out_dtype=out_dtype, want_acc=True)
    # outputs of the static variant are made here, by the caller, before the call
    y = torch.full((M, N), float("nan"), dtype=out_dtype, device="cuda")
    acc = torch.full((M, N), -1, dtype=torch.int32, device="cuda")
    torch.cuda.synchronize()
    free_before, held_before = torch.cuda.mem_get_info()[0], torch.cuda.memory_reserved()
    quest.quest_lowbit_gemm_static(xq, sx, bx, wq, sw, bw, K, y=y, acc=acc)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before, "the call changed the device's free memory"
    assert torch.cuda.memory_reserved() == held_before, "the call went through torch's allocator"
    assert quest.quest_device_status() == 0
    # the oracle decides: exact integer contraction of the same codes, then the scale product
    from oracle import quest_oracle as qo
    from tests.gpu_util import assert_output_close
    codes_x, codes_w = xq.cpu().numpy(), wq.cpu().numpy()
    ref_acc = qo.gemm_acc(codes_x, bx, codes_w, bw, K)
    assert np.array_equal(acc.cpu().numpy(), ref_acc), "int32 accumulators differ from the oracle"
    ref_y = qo.dequant(ref_acc, sx.cpu().numpy(), sw.cpu().numpy())
    assert_output_close(y.double().cpu().numpy(), ref_y, out_dtype == torch.bfloat16)
    # and the two entry points agree with each other bit for bit (same kernels, different scratch)
    assert torch.equal(acc, acc_ref), "int32 accumulators differ from quest_lowbit_gemm"
    assert torch.equal(y, y_ref), "outputs differ from quest_lowbit_gemm"


@pytest.mark.gpu
def test_static_scratch_matches_workspace_variant_on_two_calls_in_a_row():
    import paper_2502_05003_b200 as quest
    # The first call on a device looks the array's address up, and the CUDA runtime may only then load
    # the part of the library image that holds it; that one-time set-up is documented and is kept out
    # of the allocation watch by making it here, on a tiny problem.
    tiny = torch.zeros((8, 16), dtype=torch.uint8, device="cuda")
    one = torch.ones(8, device="cuda")
    quest.quest_lowbit_gemm_static(tiny, one, 4, tiny, one, 4, 32, acc=torch.empty((8, 8), dtype=torch.int32, device="cuda"))
    torch.cuda.synchronize()
    # first call nearly fills the array ((M + N) * K = 3.9 Mi bytes of int8 operands) ...
    _one_call(quest, 1000, 900, 2048, 4, 4, torch.bfloat16, seed=11)
    # ... the second is smaller, ragged and uses 8-bit codes (row sums live in the same array),
    # so any stale byte of the first call that leaked into it would change the result
    _one_call(quest, 333, 130, 1056, 8, 2, torch.float32, seed=12)
    # and the first shape once more after the array held something else
    _one_call(quest, 1000, 900, 2048, 4, 4, torch.bfloat16, seed=13)


@pytest.mark.gpu
def test_static_scratch_limit_is_reported_on_a_gpu_too():
    import paper_2502_05003_b200 as quest
    K = 4096
    xq = torch.zeros((1024, K // 2), dtype=torch.uint8, device="cuda")
    s = torch.ones(1024, device="cuda")
    y = torch.empty((1024, 1024), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(quest.QuestError) as e:          # (1024 + 1024) * 4096 = 8 Mi > 4 Mi
        quest.quest_lowbit_gemm_static(xq, s, 4, xq, s, 4, K, y=y)
    assert e.value.status == 13


def test_sizes_beyond_the_static_scratch_are_refused_on_the_host():
    """No GPU needed: the size check comes before anything touches the device."""
    from paper_2502_05003_b200 import build, _lib
    build.build()
    L = _lib.load()
    fake = ctypes.c_void_p(0x10000)
    call = lambda M, N, K, bx=4, bw=4: L.quest_lowbit_gemm_static(fake, fake, bx, fake, fake, bw, M, N, K,
                                                                  fake, 1, N, None, None)
    assert call(4096, 2048, 2048) == 13
    assert call(1 << 20, 16, 32) == 13
    assert b"static scratch" in L.quest_status_string(13)
    assert call(64, 64, 48) == 2            # K not a multiple of 32: a shape error, as in quest_lowbit_gemm
    assert call(64, 64, 128, 0, 4) == 3     # bits out of range
    assert call(16, 16, 33056, 8, 8) == 9   # would overflow int32
