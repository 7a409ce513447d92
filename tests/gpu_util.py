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
