"""Helpers for the GPU parity tests (marshalling numpy <-> torch; no method arithmetic)."""
import numpy as np
import torch


def to_dev(a: np.ndarray) -> torch.Tensor:
    """float32 stays float32; uint16 is reinterpreted as bfloat16 bit patterns."""
    t = torch.from_numpy(np.ascontiguousarray(a))
    if a.dtype == np.uint16:
        t = t.view(torch.bfloat16)
    return t.cuda()


def bf16_to_f64(t: torch.Tensor) -> np.ndarray:
    return t.float().cpu().numpy().astype(np.float64)


def guarded(shape, dtype, fill=0xAB):
    """A buffer with a canary region after it, to catch out-of-bounds writes."""
    n = int(np.prod(shape))
    itemsize = torch.empty(0, dtype=dtype).element_size()
    pad = 4096 // itemsize
    raw = torch.empty(n + pad, dtype=torch.uint8 if itemsize == 1 else dtype, device="cuda")
    raw.view(torch.uint8).fill_(fill)
    body = raw[:n].view(shape)
    return raw, body, n


def canary_intact(raw, n, fill=0xAB):
    tail = raw[n:].view(torch.uint8)
    return bool((tail == fill).all().item())


# Tolerances for outputs stored as bfloat16.  The format keeps 8 significant bits, so round-to-nearest
# costs at most half a unit in the last place = 2^-8 of the value (reached just above a power of two:
# 1 + 2^-8 lies exactly between the neighbours 1 and 1 + 2^-7), on top of the 1e-5 allowed for the
# binary32 scale product.  That bound is per element and cannot be tightened; what CAN be held to the
# 2e-3 quoted for bfloat16 data is the error of a whole output in the Euclidean norm, because the
# rounding errors of many elements average to about 2^-8 / sqrt(3) times 0.72 = 1.6e-3 of the norm.
BF16_OUT_RTOL = 2.0 ** -8 + 1e-5
BF16_OUT_NORM_RTOL = 2e-3


def assert_output_close(got, ref, out_is_bf16):
    """got, ref: float64 arrays.  Element-wise bound of the storage format plus, for bfloat16 outputs
    with enough elements for the average to mean something, the norm-wise bound."""
    tol = BF16_OUT_RTOL if out_is_bf16 else 1e-5
    bad = np.abs(got - ref) > tol * np.abs(ref) + 1e-30
    assert not bad.any(), f"{int(bad.sum())} outputs outside {tol:.2e} relative"
    if out_is_bf16 and ref.size >= 4096:
        rel = np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-300)
        assert rel <= BF16_OUT_NORM_RTOL, f"norm-wise relative error {rel:.2e}"
