"""ctypes loader for ``libquest_b200.so`` (the C ABI declared in ``include/quest.h``)."""
from __future__ import annotations

import ctypes
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libquest_b200.so")

EXPORTS = (
    "quest_quantize", "quest_trust_mask", "quest_lowbit_gemm", "quest_linear_fwd",
    "quest_workspace_bytes", "quest_codes_bytes", "quest_alpha_star", "quest_device_status", "quest_last_device_status",
    "quest_status_string", "quest_last_cuda_error", "quest_stage_timing", "quest_stage_times",
    "quest_lowbit_gemm_static", "quest_linear_bwd", "quest_bwd_workspace_bytes",
    "quest_alpha_star_fp4", "quest_quantize_fp4", "quest_lowbit_gemm_fp4", "quest_linear_fwd_fp4",
    "quest_linear_fwd_weight_only", "quest_weight_only_workspace_bytes",
    "quest_mlp_fwd", "quest_mlp_workspace_bytes", "quest_linear_fwd_quantize", "quest_linear_fwd_contract",
    "quest_selftest_bounded_wait",
)

_lib = None


class QuestError(RuntimeError):
    def __init__(self, status: int, text: str):
        super().__init__(f"quest status {status}: {text}")
        self.status = status


def load() -> ctypes.CDLL:
    """Loads the CUDA library.  There is no fallback: a missing library is an error."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2502_05003_b200.build` "
            "(nvcc, sm_100a).  This package has no CPU or PyTorch fallback.")
    L = ctypes.CDLL(LIB_PATH)
    i64, ci, cf, vp, sz = ctypes.c_int64, ctypes.c_int, ctypes.c_float, ctypes.c_void_p, ctypes.c_size_t
    L.quest_quantize.restype = ci
    L.quest_quantize.argtypes = [vp, ci, i64, i64, i64, ci, ci, cf, vp, vp, vp, vp]
    L.quest_trust_mask.restype = ci
    L.quest_trust_mask.argtypes = [vp, ci, i64, i64, i64, ci, ci, cf, vp, vp]
    L.quest_lowbit_gemm.restype = ci
    L.quest_lowbit_gemm.argtypes = [vp, vp, ci, vp, vp, ci, i64, i64, i64, vp, ci, i64, vp, vp, sz, vp]
    L.quest_lowbit_gemm_static.restype = ci
    L.quest_lowbit_gemm_static.argtypes = [vp, vp, ci, vp, vp, ci, i64, i64, i64, vp, ci, i64, vp, vp]
    L.quest_alpha_star_fp4.restype = cf
    L.quest_alpha_star_fp4.argtypes = []
    L.quest_quantize_fp4.restype = ci
    L.quest_quantize_fp4.argtypes = [vp, ci, i64, i64, i64, ci, cf, vp, vp, vp, vp]
    L.quest_lowbit_gemm_fp4.restype = ci
    L.quest_lowbit_gemm_fp4.argtypes = [vp, vp, vp, vp, i64, i64, i64, vp, ci, i64, vp, vp, sz, vp]
    L.quest_linear_fwd_fp4.restype = ci
    L.quest_linear_fwd_fp4.argtypes = [vp, vp, ci, i64, i64, i64, ci, cf, vp, ci, vp, vp, vp, vp, vp, vp, ci, vp, sz, vp]
    L.quest_linear_bwd.restype = ci
    L.quest_linear_bwd.argtypes = [vp, i64, i64, i64, ci, ci, vp, vp, vp, vp, vp, vp, vp, vp, ci, vp, sz, vp]
    L.quest_linear_fwd_weight_only.restype = ci
    L.quest_linear_fwd_weight_only.argtypes = [vp, ci, i64, vp, ci, i64, i64, i64, i64, ci, ci, cf, vp, ci, i64,
                                               vp, vp, vp, vp, vp, sz, vp]
    L.quest_weight_only_workspace_bytes.restype = sz
    L.quest_weight_only_workspace_bytes.argtypes = [i64, i64, i64]
    L.quest_bwd_workspace_bytes.restype = sz
    L.quest_bwd_workspace_bytes.argtypes = [i64, i64, i64]
    L.quest_linear_fwd.restype = ci
    L.quest_linear_fwd.argtypes = [vp, vp, ci, i64, i64, i64, ci, ci, cf, vp, ci,
                                   vp, vp, vp, vp, vp, vp, ci, vp, sz, vp]
    L.quest_linear_fwd_quantize.restype = ci
    L.quest_linear_fwd_quantize.argtypes = [vp, vp, ci, i64, i64, i64, ci, ci, cf, vp, vp, vp, vp, vp, vp, ci, vp, sz, vp]
    L.quest_linear_fwd_contract.restype = ci
    L.quest_linear_fwd_contract.argtypes = [vp, vp, i64, i64, i64, ci, vp, ci, vp, sz, vp]
    L.quest_selftest_bounded_wait.restype = ci
    L.quest_selftest_bounded_wait.argtypes = [i64, vp, vp]
    L.quest_mlp_fwd.restype = ci
    L.quest_mlp_fwd.argtypes = [vp, vp, vp, vp, ci, i64, i64, i64, ci, ci, cf, vp, vp, ci, vp, vp, sz, vp]
    L.quest_mlp_workspace_bytes.restype = sz
    L.quest_mlp_workspace_bytes.argtypes = [i64, i64, i64]
    L.quest_workspace_bytes.restype = sz
    L.quest_workspace_bytes.argtypes = [i64, i64, i64, ci, ci]
    L.quest_codes_bytes.restype = sz
    L.quest_codes_bytes.argtypes = [i64, i64, ci]
    L.quest_alpha_star.restype = cf
    L.quest_alpha_star.argtypes = [ci]
    L.quest_device_status.restype = ci
    L.quest_device_status.argtypes = [vp]
    L.quest_last_device_status.restype = ci
    L.quest_last_device_status.argtypes = [vp]
    L.quest_status_string.restype = ctypes.c_char_p
    L.quest_status_string.argtypes = [ci]
    L.quest_last_cuda_error.restype = ctypes.c_char_p
    L.quest_last_cuda_error.argtypes = []
    L.quest_stage_timing.restype = ci
    L.quest_stage_timing.argtypes = [ci]
    L.quest_stage_times.restype = ci
    L.quest_stage_times.argtypes = [vp, vp, ci]
    _lib = L
    return L


def check(status: int) -> None:
    if status != 0:
        L = load()
        text = L.quest_status_string(status).decode()
        if status == 11:
            text += " (" + L.quest_last_cuda_error().decode() + ")"
        raise QuestError(status, text)
