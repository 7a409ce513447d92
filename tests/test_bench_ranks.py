"""Host logic of the multi-rank benchmark (independent replicas, no data-path collective), run as
two gloo ranks on the CPU: max-over-ranks of the elapsed time, whole-job throughput, and the rule
that only rank 0 of `--impl reference` prints a line."""
import json
import os
import socket
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    r, w, l = bench.init_ranks(world)
    elapsed = 0.010 * (rank + 1)                   # rank 1 is the slow one
    mx = bench.max_over_ranks(elapsed, w)
    value = bench.aggregate_tokens_per_s(4096, 10, w, mx)
    with open(os.path.join(out_dir, f"rank{rank}.json"), "w") as f:
        json.dump({"rank": r, "world": w, "local": l, "max": mx, "value": value}, f)
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_take_the_slowest_time_and_sum_the_tokens(tmp_path):
    import torch.multiprocessing as mp
    port = _free_port()
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    outs = [json.load(open(tmp_path / f"rank{r}.json")) for r in range(2)]
    for r, o in enumerate(outs):
        assert o["rank"] == r and o["world"] == 2 and o["local"] == r
        assert o["max"] == pytest.approx(0.020)                       # the slower rank's time, on every rank
        assert o["value"] == pytest.approx(4096 * 10 * 2 / 0.020)     # all ranks' tokens over that time


def test_single_rank_is_the_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(0.5, 1) == 0.5
    assert bench.aggregate_tokens_per_s(100, 3, 1, 0.5) == pytest.approx(600.0)


def test_reference_arm_prints_on_rank_0_only():
    env = dict(os.environ, OMP_NUM_THREADS="2")
    base = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
            "--warmup", "0", "--ref-tokens", "16"]
    out1 = subprocess.run(base, env=dict(env, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1"), capture_output=True,
                          text=True, timeout=600)
    assert out1.returncode == 0 and out1.stdout.strip() == ""
    out0 = subprocess.run(base, env=dict(env, RANK="0", WORLD_SIZE="2", LOCAL_RANK="0"), capture_output=True,
                          text=True, timeout=600)
    assert out0.returncode == 0
    line = json.loads(out0.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "tokens/s" and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
    assert line["config"]["workload"].startswith("config 2")
