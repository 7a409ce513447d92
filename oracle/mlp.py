"""Forward pass of a Llama-style MLP block whose three linear layers are QuEST layers.

TEST INFRASTRUCTURE ONLY.  The paper's models are Llama-family transformers (hyper-parameter table:
MLP width 8/3 of the hidden size); their MLP is gate / up projection, SwiGLU, down projection, and
every linear layer of the model runs Algorithm 1.  Written out step by step:

    gate = QuEST_linear(x, w_gate)           Algorithm 1 (``quest_oracle.linear_fwd``)
    up   = QuEST_linear(x, w_up)             the same x_q for both: x is quantized once
    h    = silu(gate) * up,   silu(z) = z / (1 + exp(-z))        binary64
    y    = QuEST_linear(h16, w_down)         h16 = the hidden activations as stored (bfloat16)

READINGS.  (i) The paper does not say in which precision the hidden activations travel between
the layers; its runs use 16-bit activations, so h is rounded to bfloat16 once, after the product
silu(gate) * up, and that stored tensor is what the down projection quantizes.  (ii) gate and up are
not rounded to 16 bits on the way (they never need to leave the chip).  (iii) Rounding decisions of
the down projection depend on the stored bits of h, and an exponential evaluated in another
precision can move a bit of h; so the down projection is checked by feeding this oracle the SAME
stored h ("teacher forcing": ``down_from_hidden``), while h itself is checked against ``hidden``
within the rounding of its storage format.
Pins: tests/test_oracle_mlp.py.
"""
from __future__ import annotations

import numpy as np

from . import quest_oracle as qo


def silu(z: np.ndarray) -> np.ndarray:
    """z * sigmoid(z) in binary64, evaluated without overflow for either sign."""
    z = np.asarray(z, dtype=np.float64)
    e = np.exp(-np.abs(z))
    return np.where(z >= 0, z / (1.0 + e), z * e / (1.0 + e))


def hidden(x: np.ndarray, w_gate: np.ndarray, w_up: np.ndarray, bits: int, had_block: int,
           trust_factor: float = 1.0, rows=None) -> dict:
    """Quantize x, w_gate, w_up (Algorithm 1's rotation and projection steps), contract, dequantise,
    SwiGLU.  ``rows`` restricts the rows of x whose h is returned (sampled checks at full size); the
    quantizer outputs always cover everything."""
    K = x.shape[1]
    qx = qo.quantize(x, bits, had_block, trust_factor)
    qg = qo.quantize(w_gate, bits, had_block, trust_factor)
    qu = qo.quantize(w_up, bits, had_block, trust_factor)
    r = np.arange(x.shape[0]) if rows is None else np.sort(np.asarray(rows))
    gate = qo.dequant(qo.gemm_acc(qx["codes"][r], bits, qg["codes"], bits, K), qx["scales"][r], qg["scales"])
    up = qo.dequant(qo.gemm_acc(qx["codes"][r], bits, qu["codes"], bits, K), qx["scales"][r], qu["scales"])
    return {"h": silu(gate) * up, "gate": gate, "up": up, "x": qx, "w_gate": qg, "w_up": qu, "rows": r}


def down_from_hidden(h_bf16_bits: np.ndarray, w_down: np.ndarray, bits: int, had_block: int,
                     trust_factor: float = 1.0, rows=None) -> dict:
    """The down projection applied to the stored hidden activations (uint16 bfloat16 bit patterns)."""
    I = h_bf16_bits.shape[1]
    qh = qo.quantize(np.ascontiguousarray(h_bf16_bits), bits, had_block, trust_factor)
    qd = qo.quantize(w_down, bits, had_block, trust_factor)
    r = np.arange(h_bf16_bits.shape[0]) if rows is None else np.sort(np.asarray(rows))
    y = qo.dequant(qo.gemm_acc(qh["codes"][r], bits, qd["codes"], bits, I), qh["scales"][r], qd["scales"])
    return {"y": y, "h": qh, "w_down": qd, "rows": r}
