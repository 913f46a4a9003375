"""CPU oracle for the W4A16 linear layer (MARLIN, arxiv 2408.11743) -- TEST INFRASTRUCTURE ONLY.

Thin ctypes binding of ``marlin_oracle.c`` (plain C, fp64).  Nothing here is part
of the product: the GPU library never imports, links or calls it.  Only the test
suite, the smoke check and the benchmark's CPU-baseline leg may use it.

Array conventions (all numpy, C-contiguous):
  A          float16 [M, K]
  q_kpacked  uint32  [K/8, N]   nibble j of word (kb, n) = Q[8*kb + j, n], codes 0..15
  S          float16 [K/G, N]   G == K: one scale per output column
  C          float16 [M, N]
  2:4 form:  qc_kpacked uint32 [K/16, N] over the K/2 kept rows, idx uint8 [K/2, N] in 0..3
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "marlin_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (OpenMP, -O2, no fast-math)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-fno-fast-math",
               "-ffp-contract=off", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True, cwd=_HERE)
    return _LIB


def _load():
    global _lib
    if _lib is not None:
        return _lib
    build()
    lib = ctypes.CDLL(_LIB)
    c = ctypes
    vp = c.c_void_p
    lib.oracle_f16_to_f64.restype = c.c_double
    lib.oracle_f16_to_f64.argtypes = [c.c_uint16]
    lib.oracle_f64_to_f16.restype = c.c_uint16
    lib.oracle_f64_to_f16.argtypes = [c.c_double]
    lib.oracle_f64_to_f16_array.restype = None
    lib.oracle_f64_to_f16_array.argtypes = [vp, vp, c.c_int64]
    lib.oracle_f16_to_f64_array.restype = None
    lib.oracle_f16_to_f64_array.argtypes = [vp, vp, c.c_int64]
    lib.oracle_unpack_q.argtypes = [vp, c.c_int, c.c_int, vp]
    lib.oracle_pack_q.argtypes = [vp, c.c_int, c.c_int, vp]
    lib.oracle_dequant.argtypes = [vp, vp, c.c_int, c.c_int, c.c_int, vp]
    lib.oracle_gemm.argtypes = [vp, vp, vp, c.c_int, c.c_int, c.c_int, c.c_int, vp]
    lib.oracle_gemm_samples.argtypes = [vp, vp, vp, c.c_int, c.c_int, c.c_int, c.c_int, vp, vp, c.c_int, vp]
    lib.oracle_sparse24_expand.argtypes = [vp, vp, c.c_int, c.c_int, vp]
    lib.oracle_gemm_sparse24.argtypes = [vp, vp, vp, vp, c.c_int, c.c_int, c.c_int, c.c_int, vp]
    lib.oracle_check_tolerance.restype = c.c_int64
    lib.oracle_check_tolerance.argtypes = [vp, vp, c.c_int64, c.c_double, vp, vp]
    lib.oracle_num_threads.restype = c.c_int
    _lib = lib
    return lib


def _ptr(a: np.ndarray):
    return ctypes.c_void_p(a.ctypes.data)


def _req(a, dtype, shape=None, name="array"):
    a = np.ascontiguousarray(a)
    if a.dtype != np.dtype(dtype):
        raise TypeError(f"{name}: expected dtype {np.dtype(dtype)}, got {a.dtype}")
    if shape is not None and tuple(a.shape) != tuple(shape):
        raise ValueError(f"{name}: expected shape {tuple(shape)}, got {tuple(a.shape)}")
    return a


def _check(err: int, what: str):
    if err != 0:
        raise RuntimeError(f"oracle {what} failed with code {err}")


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def f64_to_f16(x) -> np.ndarray:
    """fp64 -> fp16 bits viewed as float16, round to nearest even, by the oracle's own routine."""
    x = np.ascontiguousarray(x, dtype=np.float64)
    out = np.empty(x.shape, dtype=np.uint16)
    _load().oracle_f64_to_f16_array(_ptr(x), _ptr(out), x.size)
    return out.view(np.float16)


def f16_to_f64(h) -> np.ndarray:
    h = _req(h, np.float16, name="h")
    out = np.empty(h.shape, dtype=np.float64)
    _load().oracle_f16_to_f64_array(_ptr(h.view(np.uint16)), _ptr(out), h.size)
    return out


def unpack_q(q_kpacked: np.ndarray) -> np.ndarray:
    """O1: canonical K-packed words -> codes Q[K, N] (uint8, 0..15)."""
    q = _req(q_kpacked, np.uint32, name="q_kpacked")
    K, N = q.shape[0] * 8, q.shape[1]
    Q = np.empty((K, N), dtype=np.uint8)
    _check(_load().oracle_unpack_q(_ptr(q), K, N, _ptr(Q)), "unpack_q")
    return Q


def pack_q(Q: np.ndarray) -> np.ndarray:
    """Inverse of unpack_q."""
    Q = _req(Q, np.uint8, name="Q")
    K, N = Q.shape
    out = np.empty((K // 8, N), dtype=np.uint32)
    _check(_load().oracle_pack_q(_ptr(Q), K, N, _ptr(out)), "pack_q")
    return out


def dequant(Q: np.ndarray, S: np.ndarray, G: int) -> np.ndarray:
    """O2: W[k, n] = (Q[k, n] - 8) * S[k // G, n] in fp64."""
    Q = _req(Q, np.uint8, name="Q")
    K, N = Q.shape
    S = _req(S, np.float16, (K // G, N), "S")
    W = np.empty((K, N), dtype=np.float64)
    _check(_load().oracle_dequant(_ptr(Q), _ptr(S.view(np.uint16)), K, N, G, _ptr(W)), "dequant")
    return W


def gemm(A: np.ndarray, q_kpacked: np.ndarray, S: np.ndarray, G: int) -> np.ndarray:
    """O1-O4: the dense W4A16 layer, fp64 accumulation, fp16 result."""
    A = _req(A, np.float16, name="A")
    M, K = A.shape
    q = _req(q_kpacked, np.uint32, name="q_kpacked")
    N = q.shape[1]
    q = _req(q, np.uint32, (K // 8, N), "q_kpacked")
    S = _req(S, np.float16, (K // G, N), "S")
    C = np.empty((M, N), dtype=np.uint16)
    _check(_load().oracle_gemm(_ptr(A.view(np.uint16)), _ptr(q), _ptr(S.view(np.uint16)), M, K, N, G, _ptr(C)),
           "gemm")
    return C.view(np.float16)


def gemm_samples(A, q_kpacked, S, G: int, ms, ns) -> np.ndarray:
    """Single outputs C[ms[i], ns[i]], each computed on its own from the packed inputs."""
    A = _req(A, np.float16, name="A")
    M, K = A.shape
    q = _req(q_kpacked, np.uint32, name="q_kpacked")
    N = q.shape[1]
    S = _req(S, np.float16, (K // G, N), "S")
    ms = np.ascontiguousarray(ms, dtype=np.int32)
    ns = np.ascontiguousarray(ns, dtype=np.int32)
    out = np.empty(ms.shape, dtype=np.uint16)
    _check(_load().oracle_gemm_samples(_ptr(A.view(np.uint16)), _ptr(q), _ptr(S.view(np.uint16)), M, K, N, G,
                                       _ptr(ms), _ptr(ns), ms.size, _ptr(out)), "gemm_samples")
    return out.view(np.float16)


def sparse24_expand(qc_kpacked: np.ndarray, idx: np.ndarray) -> np.ndarray:
    """Compressed 2:4 form -> dense codes Q[K, N] with code 8 (value 0) at pruned positions."""
    qc = _req(qc_kpacked, np.uint32, name="qc_kpacked")
    K, N = qc.shape[0] * 16, qc.shape[1]
    idx = _req(idx, np.uint8, (K // 2, N), "idx")
    Q = np.empty((K, N), dtype=np.uint8)
    _check(_load().oracle_sparse24_expand(_ptr(qc), _ptr(idx), K, N, _ptr(Q)), "sparse24_expand")
    return Q


def gemm_sparse24(A, qc_kpacked, idx, S, G: int) -> np.ndarray:
    """The 2:4 layer: expand, then O2-O4 with scale groups over the original K."""
    A = _req(A, np.float16, name="A")
    M, K = A.shape
    qc = _req(qc_kpacked, np.uint32, name="qc_kpacked")
    N = qc.shape[1]
    qc = _req(qc, np.uint32, (K // 16, N), "qc_kpacked")
    idx = _req(idx, np.uint8, (K // 2, N), "idx")
    S = _req(S, np.float16, (K // G, N), "S")
    C = np.empty((M, N), dtype=np.uint16)
    _check(_load().oracle_gemm_sparse24(_ptr(A.view(np.uint16)), _ptr(qc), _ptr(idx), _ptr(S.view(np.uint16)),
                                        M, K, N, G, _ptr(C)), "gemm_sparse24")
    return C.view(np.float16)


REL_TOL = 5e-3  # |C - C_ref| <= REL_TOL * (|C_ref| + rms(C_ref)), the acceptance bound of this build


def check_tolerance(C, C_ref, rel: float = REL_TOL):
    """Returns (failing element count, worst error/allowance ratio, rms(C_ref))."""
    C = _req(C, np.float16, name="C")
    C_ref = _req(C_ref, np.float16, C.shape, "C_ref")
    worst = ctypes.c_double(0.0)
    rms = ctypes.c_double(0.0)
    bad = _load().oracle_check_tolerance(_ptr(C.view(np.uint16)), _ptr(C_ref.view(np.uint16)), C.size, rel,
                                         ctypes.byref(worst), ctypes.byref(rms))
    return int(bad), float(worst.value), float(rms.value)
