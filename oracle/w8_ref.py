"""CPU oracle of the layer with 8-bit weights -- TEST INFRASTRUCTURE ONLY.

W[k, n] = (Q8[k, n] - 128) * S[k // G, n] (the symmetric grid of Section 3.4 with eight bits instead of four), then the
plain definition C = A . W in fp64 with numpy, rounded to fp16 once by the oracle's own conversion routine.  Also the
packed order of the codes, restated from its description: records in the order T * (K/128) + kb for the 256-column
tile T and the k-block kb; in a record, 16-byte vector c * 256 + n holds rows 128 kb + 16 c + 0..15 of column 256 T + n.
Nothing in the product imports this file.
"""
from __future__ import annotations

import numpy as np

from . import f64_to_f16


def dequant_w8(Q8: np.ndarray, S: np.ndarray, G: int) -> np.ndarray:
    K, N = Q8.shape
    assert S.shape == (K // G, N)
    return (Q8.astype(np.float64) - 128.0) * np.repeat(S.astype(np.float64), G, axis=0)


def gemm_w8(A: np.ndarray, Q8: np.ndarray, S: np.ndarray, G: int) -> np.ndarray:
    return f64_to_f16(A.astype(np.float64) @ dequant_w8(Q8, S, G))


def pack_w8(Q8: np.ndarray) -> np.ndarray:
    K, N = Q8.shape
    assert K % 128 == 0 and N % 256 == 0
    T, kb, c, n, j = np.meshgrid(np.arange(N // 256), np.arange(K // 128), np.arange(8), np.arange(256), np.arange(16),
                                 indexing="ij")
    return np.ascontiguousarray(Q8[128 * kb + 16 * c + j, 256 * T + n]).reshape(-1)
