"""CPU oracle of the gated MLP chain -- TEST INFRASTRUCTURE ONLY.

gate = fp16(A . W_gate), up = fp16(A . W_up) by the layer oracle; H = fp16(silu(gate) * up) with
silu(x) = x / (1 + exp(-x)) in fp64; C = fp16(H . W_down) by the layer oracle again.  Each step is the plain definition
(Section 3.4 for the products; the activation is the gated unit of the decoder layers whose shapes Section 5.1
benchmarks).  Nothing in the product imports this file.
"""
from __future__ import annotations

import numpy as np

from . import f64_to_f16, gemm


def silu(x: np.ndarray) -> np.ndarray:
    x = np.asarray(x, dtype=np.float64)
    return x / (1.0 + np.exp(-x))


def swiglu(gate16: np.ndarray, up16: np.ndarray) -> np.ndarray:
    """fp16 gate and up -> fp16 silu(gate) * up, one rounding."""
    return f64_to_f16(silu(gate16.astype(np.float64)) * up16.astype(np.float64))


def gate_up(A, q_gate, S_gate, q_up, S_up, G: int):
    """(gate, up, H), all fp16 [M, I]."""
    g = gemm(A, q_gate, S_gate, G)
    u = gemm(A, q_up, S_up, G)
    return g, u, swiglu(g, u)


def interleave(x_gate: np.ndarray, x_up: np.ndarray) -> np.ndarray:
    """Columns of the fused layer: blocks of 16 = eight gate columns, then the same eight up columns."""
    R, I = x_gate.shape
    out = np.empty((R, 2 * I), dtype=x_gate.dtype)
    o = out.reshape(R, I // 8, 2, 8)
    o[:, :, 0, :] = x_gate.reshape(R, I // 8, 8)
    o[:, :, 1, :] = x_up.reshape(R, I // 8, 8)
    return out
