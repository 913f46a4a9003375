"""Byte and flop accounting of the layer (Section 3.4 "Bound By Weight Loading": the product touches
16*M*K + 4*K*N + 16*M*N bits and executes M*K*N multiply-accumulates of 2 FLOPs; Section 5.1: group
scales at G = 128 add 0.125 bit per weight).  Used by the benchmark only."""
from __future__ import annotations

import json
import os


def weight_bits_fp16() -> float:
    return 16.0


def weight_bits_w4(G: int) -> float:
    return 4.0 + 16.0 / G


def weight_bytes(K: int, N: int, G: int, sparse24: bool = False, bits: int = 4) -> int:
    scales = 2 * (K // G) * N
    if bits == 8:
        return K * N + scales
    if sparse24:
        return K * N // 4 + K * N // 8 + scales
    return K * N // 2 + scales


def algorithmic_bytes(M: int, K: int, N: int, G: int, scales: bool = True, sparse24: bool = False, bits: int = 4) -> int:
    if bits == 8:
        w = weight_bytes(K, N, G, bits=8) if scales else K * N
    else:
        w = weight_bytes(K, N, G, sparse24) if scales else (K * N // 4 + K * N // 8 if sparse24 else K * N // 2)
    return w + 2 * M * K + 2 * M * N


def flops(M: int, K: int, N: int) -> int:
    return 2 * M * K * N


FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks(root: str):
    """Measured peaks (HBM copy GB/s, bf16 GEMM TFLOP/s) from MEASURED_PEAKS.json beside the benchmark, else a stated fallback."""
    path = os.path.join(root, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            d = json.load(f)
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                "source": "measured"}
    except (OSError, KeyError, ValueError):
        return dict(FALLBACK_PEAKS, source="fallback")


def roofline_seconds(M: int, K: int, N: int, G: int, peaks, sparse24: bool = False, bits: int = 4) -> float:
    t_mem = algorithmic_bytes(M, K, N, G, sparse24=sparse24, bits=bits) / (peaks["hbm_gbs"] * 1e9)
    executed = flops(M, K, N) / (2 if sparse24 else 1)
    t_flop = executed / (peaks["bf16_tflops"] * 1e12)
    return max(t_mem, t_flop)
