"""Small, bounded workloads to put under ``ncu`` (one kernel, a few launches, a few GB at most).

    python -m paper_2502_05003_b200.profile_case linear [calls]      # quest_linear_fwd, X[4096 x 2048] W[2048 x 2048], b = 4
    python -m paper_2502_05003_b200.profile_case quantize-large      # quest_quantize alone: 6144 x 5504 and 8192 x 4096
    python -m paper_2502_05003_b200.profile_case quantize-wide       # quest_quantize alone, 8192 x 4096, one rotation block per row
    python -m paper_2502_05003_b200.profile_case mlp                 # quest_mlp_fwd, 4096 tokens, H = 2048, I = 5504
    python -m paper_2502_05003_b200.profile_case backward [calls]    # quest_linear_bwd on the config-2 layer

Inputs are random (the counters of these kernels do not depend on the values); every case cycles over buffer
sets or tensors larger than L2 so that DRAM counters mean something, checks the device status word and prints
``ok``.  The summaries under ``profiles/`` name the case they were captured on.
"""
from __future__ import annotations

import sys

import torch

import paper_2502_05003_b200 as quest


def linear(calls: int = 6) -> None:
    M, K, N = 4096, 2048, 2048
    dev = torch.device("cuda")
    sets = []
    for _ in range(3):
        x = torch.randn(M, K, device=dev).bfloat16()
        w = (torch.randn(N, K, device=dev) * 0.02).bfloat16()
        sets.append((x, w, quest.alloc_workspace(M, N, K, 4, 4), quest.quest_linear_fwd(x, w, 4, 128, 1.0)))
    for i in range(calls):
        x, w, ws, out = sets[i % 3]
        quest.quest_linear_fwd(x, w, 4, 128, 1.0, y=out["y"], saved=out, workspace=ws)


def quantize_large() -> None:
    dev = torch.device("cuda")
    for rows, cols in ((6144, 5504), (8192, 4096)):
        x = torch.randn(rows, cols, device=dev).bfloat16()
        c = torch.empty(rows, cols // 2, dtype=torch.uint8, device=dev)
        s = torch.empty(rows, device=dev)
        m = torch.empty(rows, cols // 8, dtype=torch.uint8, device=dev)
        for _ in range(3):
            quest.quest_quantize(x, 4, 128, 1.0, codes=c, scales=s, mask=m)


def quantize_wide() -> None:
    dev = torch.device("cuda")
    rows, cols = 8192, 4096
    x = torch.randn(rows, cols, device=dev).bfloat16()
    c = torch.empty(rows, cols // 2, dtype=torch.uint8, device=dev)
    s = torch.empty(rows, device=dev)
    m = torch.empty(rows, cols // 8, dtype=torch.uint8, device=dev)
    for _ in range(3):
        quest.quest_quantize(x, 4, cols, 1.0, codes=c, scales=s, mask=m)


def mlp() -> None:
    T, H, I = 4096, 2048, 5504
    dev = torch.device("cuda")
    x = torch.randn(T, H, device=dev).bfloat16()
    wg = (torch.randn(I, H, device=dev) * 0.02).bfloat16()
    wu = (torch.randn(I, H, device=dev) * 0.02).bfloat16()
    wd = (torch.randn(H, I, device=dev) * 0.02).bfloat16()
    b = quest.mlp_buffers(T, H, I, 4, dev)
    for _ in range(3):
        quest.quest_mlp_fwd(x, wg, wu, wd, 4, 128, buffers=b)


def backward(calls: int = 4) -> None:
    M, K, N = 4096, 2048, 2048
    dev = torch.device("cuda")
    x = torch.randn(M, K, device=dev).bfloat16()
    w = (torch.randn(N, K, device=dev) * 0.02).bfloat16()
    fwd = quest.quest_linear_fwd(x, w, 4, 128, 1.0)
    dy = torch.randn(M, N, device=dev).bfloat16()
    for _ in range(calls):
        quest.quest_linear_bwd(dy, fwd, 4, 128, K, out_dtype=torch.bfloat16)


def main() -> None:
    if not torch.cuda.is_available():
        raise SystemExit("profile_case: needs a GPU")
    case = sys.argv[1] if len(sys.argv) > 1 else "linear"
    n = int(sys.argv[2]) if len(sys.argv) > 2 else None
    if case == "linear":
        linear(n or 6)
    elif case == "quantize-large":
        quantize_large()
    elif case == "quantize-wide":
        quantize_wide()
    elif case == "mlp":
        mlp()
    elif case == "backward":
        backward(n or 4)
    else:
        raise SystemExit(__doc__)
    torch.cuda.synchronize()
    status = quest.quest_device_status()
    if status != 0:
        raise SystemExit(f"profile_case: device status {status}")
    print("ok")


if __name__ == "__main__":
    main()
