"""CPU oracle of the quantiser front end (round to nearest with a search over clipping thresholds, Section 3.5 (a))
-- TEST INFRASTRUCTURE ONLY.  ctypes binding of ``quantize_oracle.c``; nothing in the product imports this file.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "quantize_oracle.c")
_LIB = os.path.join(_HERE, "libquantoracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile with gcc: -O2, no fast-math, no contraction of a*b+c into fused operations (the source says where it fuses)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-fno-fast-math", "-ffp-contract=off",
               "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True, cwd=_HERE)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB)
        vp, ci = ctypes.c_void_p, ctypes.c_int
        _lib.oracle_quantize_rtn.argtypes = [vp, ci, ci, ci, ci, ci, vp, vp, vp]
        _lib.oracle_quantize_rtn.restype = ci
    return _lib


def quantize_rtn(W: np.ndarray, G: int, n_grid: int = 20, n_candidates: int = 10):
    """W float16 [K, N] -> (Q uint8 [K, N] codes 0..15, S float16 [K/G, N], chosen int32 [K/G, N] candidate index)."""
    W = np.ascontiguousarray(W)
    if W.dtype != np.float16 or W.ndim != 2:
        raise TypeError("W must be float16 [K, N]")
    if not np.all(np.isfinite(W.astype(np.float32))):
        raise ValueError("W must be finite")
    K, N = W.shape
    Q = np.empty((K, N), dtype=np.uint8)
    S = np.empty((K // G, N), dtype=np.uint16)
    chosen = np.empty((K // G, N), dtype=np.int32)
    rc = _load().oracle_quantize_rtn(ctypes.c_void_p(W.ctypes.data), K, N, G, n_grid, n_candidates,
                                     ctypes.c_void_p(Q.ctypes.data), ctypes.c_void_p(S.ctypes.data),
                                     ctypes.c_void_p(chosen.ctypes.data))
    if rc != 0:
        raise ValueError("oracle_quantize_rtn: bad arguments")
    return Q, S.view(np.float16), chosen
