"""B200 (sm_100a) implementation of the QuEST quantized-linear forward pass (arXiv 2502.05003,
Algorithm 1).  This module is a thin binding over the C ABI in ``include/quest.h``: it marshals
torch tensors (device memory, current stream) into pointers and sizes; every step of the path
runs in the CUDA library.  There is no CPU or PyTorch fallback.
"""
from __future__ import annotations

import ctypes

import torch

from . import _lib
from ._lib import QuestError  # noqa: F401

F32, BF16 = 0, 1
_DT = {torch.float32: F32, torch.bfloat16: BF16}


def container_bits(bits: int) -> int:
    return 1 if bits == 1 else 2 if bits == 2 else 4 if bits <= 4 else 8


def _p(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype not in _DT:
        raise TypeError(f"unsupported dtype {t.dtype}: float32 or bfloat16")
    return _DT[t.dtype]


def _require_cuda(*ts):
    for t in ts:
        if t is not None and not t.is_cuda:
            raise ValueError("quest: tensors must live in CUDA device memory")


def quest_alpha_star(bits: int) -> float:
    return float(_lib.load().quest_alpha_star(bits))


def quest_codes_bytes(rows: int, cols: int, bits: int) -> int:
    return int(_lib.load().quest_codes_bytes(rows, cols, bits))


def quest_workspace_bytes(M: int, N: int, K: int, bits_x: int, bits_w: int) -> int:
    return int(_lib.load().quest_workspace_bytes(M, N, K, bits_x, bits_w))


def quest_device_status() -> int:
    return int(_lib.load().quest_device_status(_stream()))


def quest_last_device_status() -> int:
    return int(_lib.load().quest_last_device_status(_stream()))


def quest_selftest_bounded_wait(limit_cycles: int = 2_000_000) -> torch.Tensor:
    """Makes a bounded wait of the kernels run out on purpose (harmless: one warp, a barrier nothing completes).
    Returns the 4-int device report; afterwards ``quest_device_status()`` is 12 once, then 0."""
    report = torch.full((4,), -1, dtype=torch.int32, device="cuda")
    _lib.check(_lib.load().quest_selftest_bounded_wait(limit_cycles, _p(report), _stream()))
    return report


STAGES = ("quant_x", "quant_w", "unpack", "gemm")


def quest_stage_timing(enable: bool) -> None:
    _lib.check(_lib.load().quest_stage_timing(1 if enable else 0))


def quest_stage_times(reset=False) -> dict:
    """Collects the events of the latest call (or, for calls captured into a CUDA graph, of the
    latest replay); returns {stage: (total_ms, count)}.  ``reset``: False/0 keep the totals,
    True/1 zero them, 2 also forget stages recorded inside a capture."""
    tot = (ctypes.c_double * len(STAGES))()
    cnt = (ctypes.c_longlong * len(STAGES))()
    _lib.check(_lib.load().quest_stage_times(tot, cnt, int(reset)))
    return {name: (float(tot[i]), int(cnt[i])) for i, name in enumerate(STAGES)}


def alloc_workspace(M: int, N: int, K: int, bits_x: int, bits_w: int, device=None) -> torch.Tensor:
    n = quest_workspace_bytes(M, N, K, bits_x, bits_w)
    if n == 0:
        raise ValueError("quest: invalid GEMM shape or bit-widths")
    return torch.empty(n, dtype=torch.uint8, device=device or torch.device("cuda"))


def quest_quantize(x: torch.Tensor, bits: int, had_block: int, trust_factor: float = 1.0,
                   codes: torch.Tensor = None, scales: torch.Tensor = None, mask: torch.Tensor = None,
                   want_mask: bool = True):
    """Rows of ``x`` [rows, cols] -> (codes uint8 [rows, cols*container/8], scales f32 [rows],
    mask uint8 [rows, cols/8] or None)."""
    _require_cuda(x, codes, scales, mask)
    if x.dim() != 2 or x.stride(1) != 1:
        raise ValueError("quest_quantize: x must be 2-D with unit inner stride")
    rows, cols = x.shape
    cb = container_bits(bits) if 1 <= bits <= 8 else 8
    if codes is None:
        codes = torch.empty((rows, cols * cb // 8), dtype=torch.uint8, device=x.device)
    if scales is None:
        scales = torch.empty(rows, dtype=torch.float32, device=x.device)
    if mask is None and want_mask:
        mask = torch.empty((rows, cols // 8), dtype=torch.uint8, device=x.device)
    st = _lib.load().quest_quantize(_p(x), _dtype_code(x), rows, cols, x.stride(0), bits, had_block,
                                    ctypes.c_float(trust_factor), _p(codes), _p(scales), _p(mask), _stream())
    _lib.check(st)
    return codes, scales, mask


def quest_trust_mask(x: torch.Tensor, bits: int, had_block: int, trust_factor: float = 1.0,
                     mask: torch.Tensor = None) -> torch.Tensor:
    _require_cuda(x, mask)
    if x.dim() != 2 or x.stride(1) != 1:
        raise ValueError("quest_trust_mask: x must be 2-D with unit inner stride")
    rows, cols = x.shape
    if mask is None:
        mask = torch.empty((rows, cols // 8), dtype=torch.uint8, device=x.device)
    st = _lib.load().quest_trust_mask(_p(x), _dtype_code(x), rows, cols, x.stride(0), bits, had_block,
                                      ctypes.c_float(trust_factor), _p(mask), _stream())
    _lib.check(st)
    return mask


def quest_lowbit_gemm(xq: torch.Tensor, sx: torch.Tensor, bits_x: int,
                      wq: torch.Tensor, sw: torch.Tensor, bits_w: int, K: int,
                      out_dtype=torch.bfloat16, y: torch.Tensor = None, want_acc: bool = False,
                      acc: torch.Tensor = None, workspace: torch.Tensor = None, want_y: bool = True):
    """Packed codes -> (y [M, N] or None, acc int32 [M, N] or None)."""
    _require_cuda(xq, sx, wq, sw, y, acc, workspace)
    M, N = xq.shape[0], wq.shape[0]
    if y is None and want_y:
        y = torch.empty((M, N), dtype=out_dtype, device=xq.device)
    if acc is None and want_acc:
        acc = torch.empty((M, N), dtype=torch.int32, device=xq.device)
    if workspace is None:
        workspace = alloc_workspace(M, N, K, bits_x, bits_w, xq.device)
    st = _lib.load().quest_lowbit_gemm(_p(xq), _p(sx), bits_x, _p(wq), _p(sw), bits_w, M, N, K,
                                       _p(y), _dtype_code(y) if y is not None else 0,
                                       y.stride(0) if y is not None else N, _p(acc),
                                       _p(workspace), workspace.numel(), _stream())
    _lib.check(st)
    return y, acc


STATIC_SCRATCH_BYTES = 4 << 20


def quest_lowbit_gemm_static(xq: torch.Tensor, sx: torch.Tensor, bits_x: int,
                             wq: torch.Tensor, sw: torch.Tensor, bits_w: int, K: int,
                             y: torch.Tensor = None, acc: torch.Tensor = None):
    """``quest_lowbit_gemm`` for callers that cannot allocate: the int8 operands go to a fixed
    array inside the library instead of a workspace tensor.  The caller passes every output
    (``y`` and/or ``acc``) preallocated, so neither this wrapper nor the library allocates.
    Raises ``QuestError`` (status 13) when (M + N) * K needs more than ``STATIC_SCRATCH_BYTES``.
    Calls share the one array per device: keep them on one stream."""
    _require_cuda(xq, sx, wq, sw, y, acc)
    if y is None and acc is None:
        raise ValueError("quest_lowbit_gemm_static: pass y and/or acc preallocated")
    M, N = xq.shape[0], wq.shape[0]
    st = _lib.load().quest_lowbit_gemm_static(_p(xq), _p(sx), bits_x, _p(wq), _p(sw), bits_w, M, N, K,
                                              _p(y), _dtype_code(y) if y is not None else 0,
                                              y.stride(0) if y is not None else N, _p(acc), _stream())
    _lib.check(st)
    return y, acc


def quest_linear_fwd(x: torch.Tensor, w: torch.Tensor, bits: int, had_block: int, trust_factor: float = 1.0,
                     out_dtype=None, y: torch.Tensor = None, saved: dict = None, w_cached: dict = None,
                     workspace: torch.Tensor = None, want_masks: bool = True) -> dict:
    """Algorithm 1: returns {"y", "xq", "sx", "mx", "wq", "sw", "mw"}.

    ``saved`` may carry preallocated output tensors under those keys; ``w_cached`` = {"wq", "sw"}
    from an earlier call skips the weight quantization (then ``w`` may be None).  With
    ``w_cached["operand_in_workspace"]`` true the call also skips unpacking ``wq``: ``workspace``
    must be the tensor an earlier call for the same w used, untouched since (M may differ).
    """
    _require_cuda(x, w, y, workspace)
    M, K = x.shape
    out = dict(saved or {})
    if w_cached is not None:
        out["wq"], out["sw"] = w_cached["wq"], w_cached["sw"]
        N = out["wq"].shape[0]
    else:
        N = w.shape[0]
    cb = container_bits(bits) if 1 <= bits <= 8 else 8
    dev = x.device

    def need(key, shape, dtype):
        if out.get(key) is None:
            out[key] = torch.empty(shape, dtype=dtype, device=dev)

    need("xq", (M, K * cb // 8), torch.uint8)
    need("sx", (M,), torch.float32)
    need("wq", (N, K * cb // 8), torch.uint8)
    need("sw", (N,), torch.float32)
    if want_masks:
        need("mx", (M, K // 8), torch.uint8)
        if w_cached is None:
            need("mw", (N, K // 8), torch.uint8)
    out.setdefault("mx", None)
    out.setdefault("mw", None)
    if y is None:
        y = torch.empty((M, N), dtype=out_dtype or x.dtype, device=dev)
    if workspace is None:
        workspace = alloc_workspace(M, N, K, bits, bits, dev)
    st = _lib.load().quest_linear_fwd(
        _p(x), _p(w), _dtype_code(x), M, N, K, bits, had_block, ctypes.c_float(trust_factor),
        _p(y), _dtype_code(y), _p(out["xq"]), _p(out["sx"]), _p(out["mx"]),
        _p(out["wq"]), _p(out["sw"]), _p(out["mw"]),
        0 if w_cached is None else (2 if w_cached.get("operand_in_workspace") else 1),
        _p(workspace), workspace.numel(), _stream())
    _lib.check(st)
    out["y"] = y
    return out


def quest_linear_fwd_quantize(x: torch.Tensor, w: torch.Tensor, bits: int, had_block: int, trust_factor: float,
                              saved: dict, workspace: torch.Tensor) -> None:
    """First half of ``quest_linear_fwd``: codes, scales, masks into ``saved`` (preallocated, keys xq, sx, mx, wq,
    sw, mw) and the tensor-core operands into ``workspace``."""
    _require_cuda(x, w, workspace)
    M, K = x.shape
    N = w.shape[0]
    st = _lib.load().quest_linear_fwd_quantize(
        _p(x), _p(w), _dtype_code(x), M, N, K, bits, had_block, ctypes.c_float(trust_factor),
        _p(saved["xq"]), _p(saved["sx"]), _p(saved.get("mx")), _p(saved["wq"]), _p(saved["sw"]), _p(saved.get("mw")), 0,
        _p(workspace), workspace.numel(), _stream())
    _lib.check(st)


def quest_linear_fwd_contract(saved: dict, M: int, N: int, K: int, bits: int, y: torch.Tensor, workspace: torch.Tensor) -> None:
    """Second half of ``quest_linear_fwd``: the contraction of the operands that ``quest_linear_fwd_quantize`` left
    in ``workspace``, scaled by ``saved["sx"]`` and ``saved["sw"]``, into ``y``."""
    _require_cuda(y, workspace)
    st = _lib.load().quest_linear_fwd_contract(_p(saved["sx"]), _p(saved["sw"]), M, N, K, bits, _p(y), _dtype_code(y),
                                               _p(workspace), workspace.numel(), _stream())
    _lib.check(st)


def quest_bwd_workspace_bytes(M: int, N: int, K: int) -> int:
    return int(_lib.load().quest_bwd_workspace_bytes(M, N, K))


def quest_linear_bwd(dy: torch.Tensor, fwd: dict, bits: int, had_block: int, K: int, out_dtype=torch.float32,
                     dx: torch.Tensor = None, dw: torch.Tensor = None, want_dx: bool = True, want_dw: bool = True,
                     workspace: torch.Tensor = None) -> dict:
    """Algorithm 2 from the forward call's saved tensors (``fwd`` holds xq, sx, mx, wq, sw, mw).
    ``dy`` [M, N] bfloat16.  Returns {"dx": [M, K] or None, "dw": [N, K] or None}."""
    _require_cuda(dy, dx, dw, workspace, *[fwd[k] for k in ("xq", "sx", "mx", "wq", "sw", "mw")])
    if dy.dtype != torch.bfloat16 or not dy.is_contiguous():
        raise ValueError("quest_linear_bwd: dy must be a contiguous bfloat16 tensor")
    M, N = dy.shape
    if dx is None and want_dx:
        dx = torch.empty((M, K), dtype=out_dtype, device=dy.device)
    if dw is None and want_dw:
        dw = torch.empty((N, K), dtype=out_dtype, device=dy.device)
    if workspace is None:
        n = quest_bwd_workspace_bytes(M, N, K)
        if n == 0:
            raise ValueError("quest_linear_bwd: unsupported shape (M, N multiples of 8; K a multiple of 32, <= 16384)")
        workspace = torch.empty(n, dtype=torch.uint8, device=dy.device)
    out_t = dx if dx is not None else dw
    st = _lib.load().quest_linear_bwd(_p(dy), M, N, K, bits, had_block, _p(fwd["xq"]), _p(fwd["sx"]), _p(fwd["mx"]),
                                      _p(fwd["wq"]), _p(fwd["sw"]), _p(fwd["mw"]), _p(dx), _p(dw),
                                      _dtype_code(out_t) if out_t is not None else 0,
                                      _p(workspace), workspace.numel(), _stream())
    _lib.check(st)
    return {"dx": dx, "dw": dw}


# ---- MLP block: gate / up / SwiGLU / down, every linear layer Algorithm 1 -------------------------

class _MlpSaved(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in ("xq", "sx", "mx", "wgq", "swg", "mwg", "wuq", "swu", "mwu",
                                               "hq", "sh", "mh", "wdq", "swd", "mwd")]


def quest_mlp_workspace_bytes(T: int, H: int, I: int) -> int:
    return int(_lib.load().quest_mlp_workspace_bytes(T, H, I))


def mlp_buffers(T: int, H: int, I: int, bits: int, device=None, out_dtype=torch.bfloat16, want_masks: bool = True) -> dict:
    """Every output of ``quest_mlp_fwd`` and its workspace, allocated once (the call itself allocates nothing)."""
    dev = device or torch.device("cuda")
    cb = container_bits(bits)
    n = quest_mlp_workspace_bytes(T, H, I)
    if n == 0:
        raise ValueError("quest_mlp_fwd: unsupported shape (H, I multiples of 32, at most 16384)")
    u8 = lambda *s: torch.empty(s, dtype=torch.uint8, device=dev)
    f32 = lambda *s: torch.empty(s, dtype=torch.float32, device=dev)
    b = {"h": torch.empty((T, I), dtype=torch.bfloat16, device=dev), "y": torch.empty((T, H), dtype=out_dtype, device=dev),
         "xq": u8(T, H * cb // 8), "sx": f32(T), "wgq": u8(I, H * cb // 8), "swg": f32(I), "wuq": u8(I, H * cb // 8),
         "swu": f32(I), "hq": u8(T, I * cb // 8), "sh": f32(T), "wdq": u8(H, I * cb // 8), "swd": f32(H),
         "workspace": u8(n), "launches": 4}
    for k, shape in (("mx", (T, H // 8)), ("mwg", (I, H // 8)), ("mwu", (I, H // 8)), ("mh", (T, I // 8)), ("mwd", (H, I // 8))):
        b[k] = u8(*shape) if want_masks else None
    return b


def quest_mlp_fwd(x: torch.Tensor, w_gate: torch.Tensor, w_up: torch.Tensor, w_down: torch.Tensor, bits: int,
                  had_block: int, trust_factor: float = 1.0, buffers: dict = None, out_dtype=torch.bfloat16) -> dict:
    """y = down(silu(gate(x)) * up(x)) with QuEST linear layers.  Returns the ``buffers`` dict: "y" [T, H],
    "h" [T, I] bfloat16 and the codes / scales / masks of x, w_gate, w_up, h, w_down."""
    _require_cuda(x, w_gate, w_up, w_down)
    T, H = x.shape
    I = w_gate.shape[0]
    if w_up.shape != (I, H) or w_down.shape != (H, I) or not all(t.is_contiguous() for t in (x, w_gate, w_up, w_down)):
        raise ValueError("quest_mlp_fwd: x [T, H], w_gate / w_up [I, H], w_down [H, I], all contiguous")
    if not (x.dtype == w_gate.dtype == w_up.dtype == w_down.dtype):
        raise TypeError("quest_mlp_fwd: x and the weights share one dtype")
    b = buffers if buffers is not None else mlp_buffers(T, H, I, bits, x.device, out_dtype)
    sv = _MlpSaved(*[(b[n].data_ptr() if b.get(n) is not None else None) for n, _ in _MlpSaved._fields_])
    st = _lib.load().quest_mlp_fwd(_p(x), _p(w_gate), _p(w_up), _p(w_down), _dtype_code(x), T, H, I, bits, had_block,
                                   ctypes.c_float(trust_factor), _p(b["h"]), _p(b["y"]), _dtype_code(b["y"]),
                                   ctypes.byref(sv), _p(b["workspace"]), b["workspace"].numel(), _stream())
    _lib.check(st)
    return b


# ---- weight-only variant (Section 4.5): b-bit weights, bfloat16 activations -----------------------

def quest_weight_only_workspace_bytes(M: int, N: int, K: int) -> int:
    return int(_lib.load().quest_weight_only_workspace_bytes(M, N, K))


def quest_linear_fwd_weight_only(x: torch.Tensor, w: torch.Tensor, bits_w: int, had_block: int,
                                 trust_factor: float = 1.0, out_dtype=torch.bfloat16, out: dict = None,
                                 workspace: torch.Tensor = None) -> dict:
    """y = HT(x) (kept in bfloat16) times the quantized w.  Returns {"y", "xh", "wq", "sw", "mw"};
    ``out`` may hold preallocated tensors under those keys."""
    _require_cuda(x, w, workspace)
    if x.dim() != 2 or w.dim() != 2 or x.stride(1) != 1 or w.stride(1) != 1 or x.shape[1] != w.shape[1]:
        raise ValueError("quest_linear_fwd_weight_only: x [M, K] and w [N, K] with unit inner stride")
    M, K = x.shape
    N = w.shape[0]
    out = dict(out) if out else {}
    cb = container_bits(bits_w)

    def need(key, shape, dtype):
        if out.get(key) is None:
            out[key] = torch.empty(shape, dtype=dtype, device=x.device)
        return out[key]

    y = need("y", (M, N), out_dtype)
    xh = need("xh", (M, K), torch.bfloat16)
    wq = need("wq", (N, K * cb // 8), torch.uint8)
    sw = need("sw", (N,), torch.float32)
    mw = need("mw", (N, K // 8), torch.uint8)
    _require_cuda(y, xh, wq, sw, mw)
    if workspace is None:
        n = quest_weight_only_workspace_bytes(M, N, K)
        if n == 0:
            raise ValueError("quest_linear_fwd_weight_only: unsupported shape (K a multiple of 32, 32 <= K <= 16384)")
        workspace = torch.empty(n, dtype=torch.uint8, device=x.device)
    st = _lib.load().quest_linear_fwd_weight_only(
        _p(x), _dtype_code(x), x.stride(0), _p(w), _dtype_code(w), w.stride(0), M, N, K, bits_w, had_block,
        ctypes.c_float(trust_factor), _p(y), _dtype_code(y), y.stride(0), _p(xh), _p(wq), _p(sw), _p(mw),
        _p(workspace), workspace.numel(), _stream())
    _lib.check(st)
    return out


# ---- FP4 (E2M1) grid variant: same calls with the FP4 rounding grid of Section 4.4 ---------------

def quest_alpha_star_fp4() -> float:
    return float(_lib.load().quest_alpha_star_fp4())


def quest_quantize_fp4(x: torch.Tensor, had_block: int, trust_factor: float = 1.0):
    """Rows of ``x`` -> (E2M1 codes uint8 [rows, cols/2], scales f32 [rows], mask uint8 [rows, cols/8])."""
    _require_cuda(x)
    if x.dim() != 2 or x.stride(1) != 1:
        raise ValueError("quest_quantize_fp4: x must be 2-D with unit inner stride")
    rows, cols = x.shape
    codes = torch.empty((rows, cols // 2), dtype=torch.uint8, device=x.device)
    scales = torch.empty(rows, dtype=torch.float32, device=x.device)
    mask = torch.empty((rows, cols // 8), dtype=torch.uint8, device=x.device)
    _lib.check(_lib.load().quest_quantize_fp4(_p(x), _dtype_code(x), rows, cols, x.stride(0), had_block,
                                              ctypes.c_float(trust_factor), _p(codes), _p(scales), _p(mask), _stream()))
    return codes, scales, mask


def quest_lowbit_gemm_fp4(xq, sx, wq, sw, K: int, out_dtype=torch.bfloat16, want_acc: bool = False, workspace=None):
    """E2M1 codes -> (y [M, N], acc4 int32 [M, N] or None); acc4 is four times the value product."""
    _require_cuda(xq, sx, wq, sw, workspace)
    M, N = xq.shape[0], wq.shape[0]
    y = torch.empty((M, N), dtype=out_dtype, device=xq.device)
    acc = torch.empty((M, N), dtype=torch.int32, device=xq.device) if want_acc else None
    # the packed codes are the tensor-core operands: the call needs no scratch (the argument is kept in the ABI)
    _lib.check(_lib.load().quest_lowbit_gemm_fp4(_p(xq), _p(sx), _p(wq), _p(sw), M, N, K, _p(y), _dtype_code(y),
                                                 y.stride(0), _p(acc), _p(workspace),
                                                 workspace.numel() if workspace is not None else 0, _stream()))
    return y, acc


def quest_linear_fwd_fp4(x: torch.Tensor, w: torch.Tensor, had_block: int, trust_factor: float = 1.0,
                         out_dtype=None, w_cached: dict = None, workspace: torch.Tensor = None) -> dict:
    """Algorithm 1 with the FP4 grid: returns {"y", "xq", "sx", "mx", "wq", "sw", "mw"}."""
    _require_cuda(x, w, workspace)
    M, K = x.shape
    dev = x.device
    out = {}
    if w_cached is not None:
        out["wq"], out["sw"], out["mw"] = w_cached["wq"], w_cached["sw"], None
        N = out["wq"].shape[0]
    else:
        N = w.shape[0]
        out["wq"] = torch.empty((N, K // 2), dtype=torch.uint8, device=dev)
        out["sw"] = torch.empty(N, dtype=torch.float32, device=dev)
        out["mw"] = torch.empty((N, K // 8), dtype=torch.uint8, device=dev)
    out["xq"] = torch.empty((M, K // 2), dtype=torch.uint8, device=dev)
    out["sx"] = torch.empty(M, dtype=torch.float32, device=dev)
    out["mx"] = torch.empty((M, K // 8), dtype=torch.uint8, device=dev)
    y = torch.empty((M, N), dtype=out_dtype or x.dtype, device=dev)
    _lib.check(_lib.load().quest_linear_fwd_fp4(
        _p(x), _p(w), _dtype_code(x), M, N, K, had_block, ctypes.c_float(trust_factor), _p(y), _dtype_code(y),
        _p(out["xq"]), _p(out["sx"]), _p(out["mx"]), _p(out["wq"]), _p(out["sw"]), _p(out["mw"]),
        1 if w_cached is not None else 0, _p(workspace), workspace.numel() if workspace is not None else 0, _stream()))
    out["y"] = y
    return out
