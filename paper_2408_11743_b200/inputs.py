"""Seeded synthetic inputs for the W4A16 linear layer, shared by the tests, the
benchmark and the CPU oracle's callers.

This module holds none of the method's arithmetic: it only draws random
activations, 4-bit codes, scales and 2:4 keep-patterns with numpy and lays the
codes out in the canonical (pre-pack) input format of the library:

  q_kpacked  uint32 [K/8, N]   nibble j of word (kb, n) = code Q[8*kb + j, n], 0..15
  S          float16 [K/G, N]  G == K means one scale per output column
  2:4 form:  qc_kpacked uint32 [K/16, N] over the K/2 kept rows (same nibble rule),
             idx uint8 [K/2, N], position 0..3 of each kept value in its group of 4
             along K, strictly increasing inside each pair.

Value recipe (every config of this build): A ~ fp16(N(0,1)); codes iid uniform in
0..15 (zero point 8); scales fp16(U[0.005, 0.02]); one numpy default_rng(seed)
stream drawn in the order A, codes(, keep patterns), scales.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Iterator, Tuple

import numpy as np


def kpack(Q: np.ndarray) -> np.ndarray:
    """Codes [K, N] (0..15) -> canonical words [K/8, N]; low nibble = lowest k."""
    K, N = Q.shape
    assert K % 8 == 0
    q = Q.astype(np.uint32).reshape(K // 8, 8, N)
    out = np.zeros((K // 8, N), dtype=np.uint32)
    for j in range(8):
        out |= q[:, j, :] << np.uint32(4 * j)
    return out


@dataclass
class DenseCase:
    A: np.ndarray          # float16 [M, K]
    q_kpacked: np.ndarray  # uint32 [K/8, N]
    S: np.ndarray          # float16 [K/G, N]
    M: int
    K: int
    N: int
    G: int
    seed: int


@dataclass
class SparseCase:
    A: np.ndarray           # float16 [M, K]
    qc_kpacked: np.ndarray  # uint32 [K/16, N]
    idx: np.ndarray         # uint8 [K/2, N]
    S: np.ndarray           # float16 [K/G, N]
    M: int
    K: int
    N: int
    G: int
    seed: int


def _draw_A(rng, M, K):
    return rng.standard_normal((M, K), dtype=np.float32).astype(np.float16)


def _draw_S(rng, K, N, G):
    return rng.uniform(0.005, 0.02, size=(K // G, N)).astype(np.float16)


def make_dense(M: int, K: int, N: int, G: int, seed: int) -> DenseCase:
    if G in (-1, 0):
        G = K
    rng = np.random.default_rng(seed)
    A = _draw_A(rng, M, K)
    Q = rng.integers(0, 16, size=(K, N), dtype=np.uint8)
    S = _draw_S(rng, K, N, G)
    return DenseCase(A, kpack(Q), S, M, K, N, G, seed)


# the six ways of keeping two of four, as (first, second) positions
_KEEP_PATTERNS = np.array([(0, 1), (0, 2), (0, 3), (1, 2), (1, 3), (2, 3)], dtype=np.uint8)


def make_sparse24(M: int, K: int, N: int, G: int, seed: int) -> SparseCase:
    if G in (-1, 0):
        G = K
    assert K % 16 == 0
    rng = np.random.default_rng(seed)
    A = _draw_A(rng, M, K)
    Qc = rng.integers(0, 16, size=(K // 2, N), dtype=np.uint8)
    pat = rng.integers(0, 6, size=(K // 4, N))
    idx = np.empty((K // 2, N), dtype=np.uint8)
    idx[0::2, :] = _KEEP_PATTERNS[pat, 0]
    idx[1::2, :] = _KEEP_PATTERNS[pat, 1]
    S = _draw_S(rng, K, N, G)
    return SparseCase(A, kpack(Qc), idx, S, M, K, N, G, seed)


# ---- the workloads of this build (synthetic stand-ins for the paper's layer benchmarks) ----

LLAMA7B_LAYERS = [("qkv", 4096, 12288), ("o_proj", 4096, 4096), ("gate_up", 4096, 22016), ("down", 11008, 4096)]
LLAMA70B_LAYERS = [("gate_up", 8192, 57344), ("down", 28672, 8192), ("skinny", 28672, 1024)]


def case_seed(config: int, layer_index: int, M: int, per_channel: bool = False) -> int:
    return 100000 * config + 1000 * layer_index + M + (500 if per_channel else 0)


def iter_cases(config: int) -> Iterator[Tuple[str, int, int, int, int, int]]:
    """Yields (layer name, M, K, N, G, seed) for one of the five workload configs."""
    if config == 1:
        yield ("single", 16, 4096, 4096, 128, 0)
    elif config == 2:
        for M in (1, 2, 4, 8, 16, 32, 64, 128):
            yield ("sweep", M, 8192, 8192, 128, case_seed(2, 0, M))
    elif config == 3:
        for li, (name, K, N) in enumerate(LLAMA7B_LAYERS):
            for M in (1, 16, 32, 64, 128):
                yield (name, M, K, N, 128, case_seed(3, li, M))
    elif config == 4:
        for li, (name, K, N) in enumerate(LLAMA70B_LAYERS):
            for G in (K, 128):
                for M in (1, 16, 64, 128):
                    yield (name, M, K, N, G, case_seed(4, li, M, per_channel=(G == K)))
    elif config == 5:
        for M in (16, 32, 64, 128):
            yield ("sparse24", M, 8192, 8192, 128, case_seed(5, 0, M))
    else:
        raise ValueError(f"unknown config {config}")
