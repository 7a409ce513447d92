"""The bounded waits of the kernels: their time-out path, run on purpose and without any fault.

A one-warp self-test kernel of the library waits, with a limit of about a millisecond, on a barrier that nothing
completes, through the same wait routine the tensor-core kernels use.  The wait must give up and return (the
kernel ends by itself), the status word must report the time-out exactly once, and the library must work
normally afterwards.
"""
import numpy as np
import pytest
import torch

from oracle import quest_oracle as qo
from tests.helpers import container_bits

pytestmark = pytest.mark.gpu


def test_a_wait_that_runs_out_is_reported_once_and_leaves_the_context_usable():
    import paper_2502_05003_b200 as quest
    assert quest.quest_device_status() == 0
    report = quest.quest_selftest_bounded_wait(2_000_000)        # about a millisecond of SM clock cycles
    torch.cuda.synchronize()                                      # the kernel returns by itself
    assert report.cpu().tolist() == [0, 0, 1, 1]                  # gave up; refused at once; abort raised; second wait short
    assert quest.quest_device_status() == 12                      # QUEST_ERR_DEVICE_TIMEOUT, read and cleared
    assert quest.quest_device_status() == 0
    assert quest.quest_last_device_status() == 0
    # a normal contraction afterwards is bit-exact
    rng = np.random.default_rng(0)
    M, N, K = 128, 128, 128
    cb = container_bits(4)
    xq = rng.integers(0, 256, size=(M, K * cb // 8), dtype=np.uint8)
    wq = rng.integers(0, 256, size=(N, K * cb // 8), dtype=np.uint8)
    d = lambda a: torch.from_numpy(a).cuda()
    ones = torch.ones(M, device="cuda")
    _, acc = quest.quest_lowbit_gemm(d(xq), ones, 4, d(wq), ones, 4, K, want_acc=True)
    torch.cuda.synchronize()
    assert np.array_equal(acc.cpu().numpy(), qo.gemm_acc(xq, 4, wq, 4, K))
    assert quest.quest_device_status() == 0


def test_limits_outside_the_documented_range_are_refused_on_the_host():
    import paper_2502_05003_b200 as quest
    for bad in (0, 999, 5_000_000_000):
        with pytest.raises(quest.QuestError):
            quest.quest_selftest_bounded_wait(bad)
    assert quest.quest_device_status() == 0
