"""ctypes loader for ``quest_oracle.c`` (the canonical binary32 oracle).

TEST INFRASTRUCTURE ONLY.  Builds the C file with gcc on first use (into ``oracle/_build``)
and exposes thin numpy wrappers; every numeric step lives in the C file.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "quest_oracle.c")
_BUILD = os.path.join(_HERE, "_build")
_LIB_PATH = os.path.join(_BUILD, "libquest_oracle.so")
_lock = threading.Lock()
_lib = None

F32, BF16 = 0, 1


def build(force: bool = False) -> str:
    """Compile the oracle (gcc, OpenMP, no FMA contraction, no fast-math)."""
    os.makedirs(_BUILD, exist_ok=True)
    if force or not os.path.exists(_LIB_PATH) or os.path.getmtime(_LIB_PATH) < os.path.getmtime(_SRC):
        tmp = _LIB_PATH + f".{os.getpid()}.tmp"
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-ffp-contract=off", "-fno-fast-math", "-shared", "-fPIC",
             "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB_PATH)
    return _LIB_PATH


def lib() -> ctypes.CDLL:
    global _lib
    with _lock:
        if _lib is None:
            L = ctypes.CDLL(build())
            i64, c_int, c_float, vp = ctypes.c_int64, ctypes.c_int, ctypes.c_float, ctypes.c_void_p
            L.qo_alpha_star.restype = c_float
            L.qo_alpha_star.argtypes = [c_int]
            L.qo_container_bits.restype = c_int
            L.qo_container_bits.argtypes = [c_int]
            L.qo_fwht_block.restype = None
            L.qo_fwht_block.argtypes = [vp, c_int]
            L.qo_quantize.restype = c_int
            L.qo_quantize.argtypes = [vp, c_int, i64, i64, i64, c_int, c_int, c_float, vp, vp, vp, vp, vp]
            L.qo_unpack_grid_values.restype = c_int
            L.qo_unpack_grid_values.argtypes = [vp, i64, i64, c_int, vp]
            L.qo_gemm_acc.restype = c_int
            L.qo_gemm_acc.argtypes = [vp, c_int, vp, c_int, i64, i64, i64, vp]
            L.qo_dequant.restype = c_int
            L.qo_dequant.argtypes = [vp, vp, vp, i64, i64, vp]
            L.qo_linear_fwd.restype = c_int
            L.qo_linear_fwd.argtypes = [vp, vp, c_int, i64, i64, i64, c_int, c_int, c_float,
                                        vp, vp, vp, vp, vp, vp, vp, vp]
            L.qo_e2m1_code.restype = c_int
            L.qo_e2m1_code.argtypes = [c_float]
            L.qo_alpha_star_fp4.restype = c_float
            L.qo_alpha_star_fp4.argtypes = []
            L.qo_quantize_fp4.restype = c_int
            L.qo_quantize_fp4.argtypes = [vp, c_int, i64, i64, i64, c_int, c_float, vp, vp, vp, vp]
            L.qo_unpack_fp4_twice.restype = c_int
            L.qo_unpack_fp4_twice.argtypes = [vp, i64, i64, vp]
            L.qo_gemm_acc_fp4.restype = c_int
            L.qo_gemm_acc_fp4.argtypes = [vp, vp, i64, i64, i64, vp]
            _lib = L
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _check(st, what):
    if st != 0:
        raise ValueError(f"oracle {what} failed with status {st}")


def _dtype_code(x: np.ndarray) -> int:
    if x.dtype == np.float32:
        return F32
    if x.dtype == np.uint16:  # bfloat16 bit patterns
        return BF16
    raise TypeError("x must be float32 or uint16 (bfloat16 bits)")


def alpha_star(bits: int) -> float:
    return float(lib().qo_alpha_star(bits))


def container_bits(bits: int) -> int:
    return int(lib().qo_container_bits(bits))


def fwht_block(v: np.ndarray) -> np.ndarray:
    out = np.ascontiguousarray(v, dtype=np.float32).copy()
    lib().qo_fwht_block(_ptr(out), out.size)
    return out


def quantize(x: np.ndarray, bits: int, had_block: int, trust_factor: float = 1.0,
             want_mask: bool = True, debug: bool = False) -> dict:
    """Rows of ``x`` (float32, or uint16 holding bfloat16 bits) -> codes, scales, mask."""
    assert x.ndim == 2
    x = np.ascontiguousarray(x)
    rows, cols = x.shape
    cb = container_bits(bits)
    codes = np.zeros((rows, cols * cb // 8), np.uint8)
    scales = np.zeros(rows, np.float32)
    mask = np.zeros((rows, cols // 8), np.uint8) if want_mask else None
    u = np.zeros((rows, cols), np.float32) if debug else None
    t = np.zeros((rows, cols), np.float32) if debug else None
    st = lib().qo_quantize(_ptr(x), _dtype_code(x), rows, cols, cols, bits, had_block,
                           ctypes.c_float(trust_factor), _ptr(codes), _ptr(scales), _ptr(mask),
                           _ptr(u), _ptr(t))
    _check(st, "quantize")
    out = {"codes": codes, "scales": scales, "mask": mask}
    if debug:
        out["u"], out["t"] = u, t
    return out


def unpack_grid_values(codes: np.ndarray, cols: int, bits: int) -> np.ndarray:
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    rows = codes.shape[0]
    c = np.zeros((rows, cols), np.int16)
    _check(lib().qo_unpack_grid_values(_ptr(codes), rows, cols, bits, _ptr(c)), "unpack")
    return c


def gemm_acc(xq: np.ndarray, bits_x: int, wq: np.ndarray, bits_w: int, K: int) -> np.ndarray:
    xq = np.ascontiguousarray(xq, dtype=np.uint8)
    wq = np.ascontiguousarray(wq, dtype=np.uint8)
    M, N = xq.shape[0], wq.shape[0]
    acc = np.zeros((M, N), np.int32)
    _check(lib().qo_gemm_acc(_ptr(xq), bits_x, _ptr(wq), bits_w, M, N, K, _ptr(acc)), "gemm_acc")
    return acc


def dequant(acc: np.ndarray, sx: np.ndarray, sw: np.ndarray) -> np.ndarray:
    acc = np.ascontiguousarray(acc, dtype=np.int32)
    sx = np.ascontiguousarray(sx, dtype=np.float32)
    sw = np.ascontiguousarray(sw, dtype=np.float32)
    M, N = acc.shape
    y = np.zeros((M, N), np.float64)
    _check(lib().qo_dequant(_ptr(acc), _ptr(sx), _ptr(sw), M, N, _ptr(y)), "dequant")
    return y


def linear_fwd(x: np.ndarray, w: np.ndarray, bits: int, had_block: int,
               trust_factor: float = 1.0) -> dict:
    x = np.ascontiguousarray(x)
    w = np.ascontiguousarray(w)
    assert x.dtype == w.dtype and x.shape[1] == w.shape[1]
    M, K = x.shape
    N = w.shape[0]
    cb = container_bits(bits)
    out = {
        "y": np.zeros((M, N), np.float64), "acc": np.zeros((M, N), np.int32),
        "xq": np.zeros((M, K * cb // 8), np.uint8), "sx": np.zeros(M, np.float32),
        "mx": np.zeros((M, K // 8), np.uint8),
        "wq": np.zeros((N, K * cb // 8), np.uint8), "sw": np.zeros(N, np.float32),
        "mw": np.zeros((N, K // 8), np.uint8),
    }
    st = lib().qo_linear_fwd(_ptr(x), _ptr(w), _dtype_code(x), M, N, K, bits, had_block,
                             ctypes.c_float(trust_factor), _ptr(out["y"]), _ptr(out["acc"]),
                             _ptr(out["xq"]), _ptr(out["sx"]), _ptr(out["mx"]),
                             _ptr(out["wq"]), _ptr(out["sw"]), _ptr(out["mw"]))
    _check(st, "linear_fwd")
    return out


# ---- FP4 (E2M1) grid variant ---------------------------------------------------------------------

def alpha_star_fp4() -> float:
    return float(lib().qo_alpha_star_fp4())


def e2m1_code(t: float) -> int:
    return int(lib().qo_e2m1_code(ctypes.c_float(t)))


def quantize_fp4(x: np.ndarray, had_block: int, trust_factor: float = 1.0, debug: bool = False) -> dict:
    """Rows of ``x`` -> E2M1 codes (two per byte), scales (xq_h = scale * E2M1 value), trust mask."""
    x = np.ascontiguousarray(x)
    rows, cols = x.shape
    codes = np.zeros((rows, cols // 2), np.uint8)
    scales = np.zeros(rows, np.float32)
    mask = np.zeros((rows, cols // 8), np.uint8)
    t = np.zeros((rows, cols), np.float32) if debug else None
    _check(lib().qo_quantize_fp4(_ptr(x), _dtype_code(x), rows, cols, cols, had_block, ctypes.c_float(trust_factor),
                                 _ptr(codes), _ptr(scales), _ptr(mask), _ptr(t)), "quantize_fp4")
    out = {"codes": codes, "scales": scales, "mask": mask}
    if debug:
        out["t"] = t
    return out


def unpack_fp4_twice(codes: np.ndarray, cols: int) -> np.ndarray:
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    c2 = np.zeros((codes.shape[0], cols), np.int16)
    _check(lib().qo_unpack_fp4_twice(_ptr(codes), codes.shape[0], cols, _ptr(c2)), "unpack_fp4")
    return c2


def gemm_acc_fp4(xq: np.ndarray, wq: np.ndarray, K: int) -> np.ndarray:
    """acc4 = sum_k (2 v_x)(2 v_w): four times the product of the E2M1 values, exact int32."""
    xq = np.ascontiguousarray(xq, dtype=np.uint8)
    wq = np.ascontiguousarray(wq, dtype=np.uint8)
    acc = np.zeros((xq.shape[0], wq.shape[0]), np.int32)
    _check(lib().qo_gemm_acc_fp4(_ptr(xq), _ptr(wq), xq.shape[0], wq.shape[0], K, _ptr(acc)), "gemm_acc_fp4")
    return acc


def dequant_fp4(acc4: np.ndarray, sx: np.ndarray, sw: np.ndarray) -> np.ndarray:
    return np.asarray(sx, np.float64)[:, None] * np.asarray(sw, np.float64)[None, :] * np.asarray(acc4, np.float64) / 4.0
