"""CPU oracle of the layer with zero points -- TEST INFRASTRUCTURE ONLY.

Section 2.3 quantises a group as q = round((v - z) / s) with a zero point and a scale per group; with an integer zero
point the reconstruction is W[k, n] = (Q[k, n] - Z[k // G, n]) * S[k // G, n].  The layer is then the plain definition
C = A . W, written out with numpy in fp64 and rounded to fp16 once by the oracle's own conversion routine.  Nothing in
the product imports this file.
"""
from __future__ import annotations

import numpy as np

from . import f64_to_f16, unpack_q


def dequant_zp(Q: np.ndarray, S: np.ndarray, Z: np.ndarray, G: int) -> np.ndarray:
    """W[k, n] = (Q[k, n] - Z[k // G, n]) * S[k // G, n] in fp64."""
    K, N = Q.shape
    assert S.shape == (K // G, N) and Z.shape == (K // G, N)
    return (Q.astype(np.float64) - np.repeat(Z.astype(np.float64), G, axis=0)) * np.repeat(S.astype(np.float64), G, axis=0)


def gemm_zp(A: np.ndarray, q_kpacked: np.ndarray, S: np.ndarray, Z: np.ndarray, G: int) -> np.ndarray:
    """C = A . W in fp64, rounded to fp16 (nearest even)."""
    Q = unpack_q(q_kpacked)
    W = dequant_zp(Q, S, Z, G)
    return f64_to_f16(A.astype(np.float64) @ W)
