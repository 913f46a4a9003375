"""B200-native W4A16 linear layer (the hot path of MARLIN, arxiv 2408.11743).

The product is the C-ABI library ``libmarlin_b200.so`` declared in ``include/marlin_b200.h``;
``binding`` marshals torch device tensors into it.  Nothing is loaded at import time; the first
call loads the library and raises if it is missing (there is no CPU or eager fallback).
"""
from .binding import (  # noqa: F401
    Layer,
    MarlinError,
    gemm,
    gemm_sparse24,
    gemm_static_ws,
    gemm_swiglu,
    gemm_w8,
    interleave_gate_up,
    gemm_zp,
    lib,
    mlp_swiglu,
    library_path,
    new_workspace,
    pack,
    pack_sparse24,
    pack_w8,
    pack_zeros,
    plan_stripes,
    quantize_rtn,
    read_status,
    unpack,
    unpack_sparse24,
    unpack_w8,
    unpack_zeros,
    workspace_bytes,
)
