"""Bit-width and shape sweep of the two kernels: ``python -m paper_2502_05003_b200.sweep [--quick]``.

For every point (b, d, tokens, g) of the sweep (bf16 Student-t(4) activations X[tokens x d], square
weights W[d x d] ~ N(0, 0.02^2), seeded) it reports the quantizer's achieved GB/s on X (algorithmic
bytes: input + codes + mask + scales) and the low-bit GEMM's TOP/s (2 M N K) on [tokens x d] x [d x d].
Timing: CUDA events; the quantizer is replayed from a CUDA graph over a ring of buffers larger than
L2, the GEMM stage is timed by event nodes inside a graph.  Prints one JSON object per point and a
markdown table at the end.
"""
from __future__ import annotations

import argparse
import json
import os

import torch

from . import (alloc_workspace, container_bits, quest_lowbit_gemm, quest_quantize, quest_stage_times,
               quest_stage_timing, synth)

L2_BYTES = 126 << 20


def _graph_time_us(fn, nset: int, reps: int) -> float:
    for i in range(max(3, nset)):
        fn(i)
    torch.cuda.synchronize()
    st = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(st):
        with torch.cuda.graph(g, stream=st):
            for i in range(nset):
                fn(i)
    g.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        g.replay()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) * 1e3 / (reps * nset)


def run_point(index: int, bits: int, d: int, tokens: int, g: int, hbm_gbs: float, int8_tops: float) -> dict:
    dev = torch.device("cuda")
    p = synth.config5_point(index, tokens, d)
    x = torch.from_numpy(p["x"]).view(torch.bfloat16).to(dev)
    w = torch.from_numpy(p["w"]).view(torch.bfloat16).to(dev)
    cb = container_bits(bits)
    q_bytes = tokens * d * (2 + cb / 8 + 1 / 8) + 4 * tokens
    nset = max(2, int(3 * L2_BYTES / q_bytes) + 1)
    sets = [(x.clone(), torch.empty(tokens, d * cb // 8, dtype=torch.uint8, device=dev),
             torch.empty(tokens, device=dev), torch.empty(tokens, d // 8, dtype=torch.uint8, device=dev))
            for _ in range(nset)]

    def qfn(i):
        xi, c, s, m = sets[i % nset]
        quest_quantize(xi, bits, g, 1.0, codes=c, scales=s, mask=m)

    q_us = _graph_time_us(qfn, nset, max(1, 200 // nset))
    xq, sx, _ = quest_quantize(x, bits, g)
    wq, sw, _ = quest_quantize(w, bits, g)
    del sets
    g_bytes = tokens * d + d * d + tokens * d * 2
    gset = max(2, int(3 * L2_BYTES / g_bytes) + 1)
    gsets = [(xq.clone(), wq.clone(), torch.empty(tokens, d, dtype=torch.bfloat16, device=dev),
              alloc_workspace(tokens, d, d, bits, bits)) for _ in range(gset)]

    def gfn(i):
        a, b, y, ws = gsets[i % gset]
        quest_lowbit_gemm(a, sx, bits, b, sw, bits, d, y=y, workspace=ws)

    for i in range(3):
        gfn(i)
    quest_stage_timing(True)
    quest_stage_times(reset=2)
    st = torch.cuda.Stream()
    gg = torch.cuda.CUDAGraph()
    with torch.cuda.stream(st):
        with torch.cuda.graph(gg, stream=st):
            for i in range(gset):
                gfn(i)
    for _ in range(20):
        gg.replay()
        quest_stage_times()
    stage = quest_stage_times(reset=2)
    quest_stage_timing(False)
    g_us = stage["gemm"][0] / stage["gemm"][1] * 1e3
    tops = 2.0 * tokens * d * d / g_us / 1e6
    gbs = q_bytes / q_us / 1e3
    # one- and two-bit codes run on the FP4 tensor-core path: nominal rate twice that of int8
    path, peak = ("mxf4", 2.0 * int8_tops) if bits <= 2 else ("i8", int8_tops)
    return {"bits": bits, "d": d, "tokens": tokens, "g": g, "quant_us": round(q_us, 2), "quant_GBps": round(gbs, 1),
            "quant_frac_hbm": round(gbs / hbm_gbs, 3), "gemm_us": round(g_us, 2), "gemm_TOPS": round(tops, 1),
            "gemm_path": path, "gemm_frac_peak": round(tops / peak, 3)}


def measured_peaks():
    """Denominators: MEASURED_PEAKS.json at the repository root (HBM copy rate; int8 tensor rate taken as twice the
    measured bf16 burst rate, the nominal ratio), else the stated fallback figures."""
    path = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return float(p["hbm_gbs"]), 2.0 * float(p["bf16_tflops"]), "measured"
    return 6650.0, 2.0 * 1590.0, "fallback"


def main():
    hbm, int8, source = measured_peaks()
    ap = argparse.ArgumentParser()
    ap.add_argument("--quick", action="store_true", help="b = 4 only")
    ap.add_argument("--hbm-gbs", type=float, default=hbm, help="HBM copy rate (denominator; default: %s)" % source)
    ap.add_argument("--int8-tops", type=float, default=int8, help="2 x bf16 burst rate (denominator; default: %s)" % source)
    args = ap.parse_args()
    print(json.dumps({"denominators": {"hbm_gbs": args.hbm_gbs, "int8_tops": args.int8_tops, "source": source}}), flush=True)
    rows = []
    index = 0
    for bits in ((4,) if args.quick else (1, 2, 3, 4, 8)):
        for d in (512, 1024, 2048, 4096):
            for tokens in (1024, 16384):
                for g in (128, d):
                    r = run_point(index, bits, d, tokens, g, args.hbm_gbs, args.int8_tops)
                    index += 1
                    rows.append(r)
                    print(json.dumps(r), flush=True)
    print("\n| b | d | tokens | g | quantizer us | GB/s | of HBM | GEMM path | GEMM us | TOP/s | of its peak |")
    print("|---|---|---|---|---:|---:|---:|---|---:|---:|---:|")
    for r in rows:
        print(f"| {r['bits']} | {r['d']} | {r['tokens']} | {r['g']} | {r['quant_us']} | {r['quant_GBps']} | "
              f"{r['quant_frac_hbm']} | {r['gemm_path']} | {r['gemm_us']} | {r['gemm_TOPS']} | {r['gemm_frac_peak']} |")


if __name__ == "__main__":
    main()
