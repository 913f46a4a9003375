"""ctypes binding of libmarlin_b200.so: same names as the C ABI, argument marshalling only.

Every step of the layer (re-layout, streaming, dequantisation, tensor-core product, stripe
fix-up) runs inside the library's CUDA kernels.  torch is used for device memory and streams.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libmarlin_b200.so")
_lib = None

EXPORTS = [
    "marlin_status_string", "marlin_packed_weight_bytes", "marlin_packed_scale_bytes", "marlin_packed_meta_bytes",
    "marlin_workspace_bytes", "marlin_pack", "marlin_unpack", "marlin_gemm", "marlin_pack_sparse24",
    "marlin_unpack_sparse24", "marlin_gemm_sparse24", "marlin_read_status", "marlin_plan_stripes",
    "marlin_gemm_static_ws", "marlin_quantize_rtn", "marlin_pack_zeros", "marlin_unpack_zeros", "marlin_gemm_zp",
    "marlin_interleave_gate_up", "marlin_gemm_swiglu", "marlin_mlp_swiglu",
    "marlin_packed_weight_bytes_w8", "marlin_pack_w8", "marlin_unpack_w8", "marlin_gemm_w8",
]
STATIC_WS_MAX_M = 16  # MARLIN_STATIC_WS_MAX_M of the header


class MarlinError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        msg = lib().marlin_status_string(status).decode()
        super().__init__(f"{what}: marlin status {status} ({msg})")


def library_path() -> str:
    return _LIB_PATH


def lib():
    """Loads the shared library (once).  Raises if it has not been built: no fallback exists."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise RuntimeError(
            f"{_LIB_PATH} is missing: build it with `python -m paper_2408_11743_b200.build` "
            "(this package has no CPU or eager path)")
    L = ctypes.CDLL(_LIB_PATH)
    c = ctypes
    vp, i, sz = c.c_void_p, c.c_int, c.c_size_t
    L.marlin_status_string.restype = c.c_char_p
    L.marlin_status_string.argtypes = [i]
    L.marlin_packed_weight_bytes.restype = sz
    L.marlin_packed_weight_bytes.argtypes = [i, i, i]
    L.marlin_packed_scale_bytes.restype = sz
    L.marlin_packed_scale_bytes.argtypes = [i, i, i]
    L.marlin_packed_meta_bytes.restype = sz
    L.marlin_packed_meta_bytes.argtypes = [i, i]
    L.marlin_workspace_bytes.restype = sz
    L.marlin_workspace_bytes.argtypes = [i, i, i]
    L.marlin_pack.argtypes = [vp, vp, vp, vp, i, i, i, vp]
    L.marlin_unpack.argtypes = [vp, vp, vp, vp, i, i, i, vp]
    L.marlin_quantize_rtn.argtypes = [vp, vp, vp, i, i, i, i, i, vp]
    L.marlin_pack_zeros.argtypes = [vp, vp, i, i, i, vp]
    L.marlin_unpack_zeros.argtypes = [vp, vp, i, i, i, vp]
    L.marlin_gemm_zp.argtypes = [vp, vp, vp, vp, vp, i, i, i, i, vp, sz, vp]
    L.marlin_packed_weight_bytes_w8.restype = sz
    L.marlin_packed_weight_bytes_w8.argtypes = [i, i]
    L.marlin_pack_w8.argtypes = [vp, vp, vp, vp, i, i, i, vp]
    L.marlin_unpack_w8.argtypes = [vp, vp, vp, vp, i, i, i, vp]
    L.marlin_gemm_w8.argtypes = [vp, vp, vp, vp, i, i, i, i, vp, sz, vp]
    L.marlin_interleave_gate_up.argtypes = [vp, vp, vp, vp, vp, vp, i, i, i, vp]
    L.marlin_gemm_swiglu.argtypes = [vp, vp, vp, vp, i, i, i, i, vp, sz, vp]
    L.marlin_mlp_swiglu.argtypes = [vp, vp, vp, vp, vp, vp, vp, i, i, i, i, i, vp, sz, vp]
    L.marlin_gemm.argtypes = [vp, vp, vp, vp, i, i, i, i, vp, sz, vp]
    L.marlin_gemm_static_ws.argtypes = [vp, vp, vp, vp, i, i, i, i, vp]
    L.marlin_pack_sparse24.argtypes = [vp, vp, vp, vp, vp, vp, i, i, i, vp]
    L.marlin_unpack_sparse24.argtypes = [vp, vp, vp, vp, vp, vp, i, i, i, vp]
    L.marlin_gemm_sparse24.argtypes = [vp, vp, vp, vp, vp, i, i, i, i, vp, sz, vp]
    L.marlin_read_status.argtypes = [vp, vp]
    L.marlin_plan_stripes.argtypes = [i, i, i, i, vp, vp, vp, i]
    for name in ("marlin_pack_w8", "marlin_unpack_w8", "marlin_gemm_w8", "marlin_interleave_gate_up", "marlin_gemm_swiglu", "marlin_mlp_swiglu", "marlin_pack_zeros", "marlin_unpack_zeros", "marlin_gemm_zp", "marlin_quantize_rtn", "marlin_gemm_static_ws", "marlin_pack", "marlin_unpack", "marlin_gemm", "marlin_pack_sparse24", "marlin_unpack_sparse24",
                 "marlin_gemm_sparse24", "marlin_read_status", "marlin_plan_stripes"):
        getattr(L, name).restype = i
    _lib = L
    return L


def _torch():
    import torch
    return torch


def _stream_ptr(stream=None) -> int:
    torch = _torch()
    s = stream if stream is not None else torch.cuda.current_stream()
    return int(s.cuda_stream)


def _dev(t, dtype, name):
    torch = _torch()
    if not isinstance(t, torch.Tensor) or not t.is_cuda:
        raise TypeError(f"{name} must be a CUDA tensor")
    if t.dtype != dtype:
        raise TypeError(f"{name} must have dtype {dtype}, got {t.dtype}")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    return t


def _check(status: int, what: str):
    if status != 0:
        raise MarlinError(status, what)


def workspace_bytes(max_M: int, K: int, N: int) -> int:
    n = int(lib().marlin_workspace_bytes(max_M, K, N))
    if n == 0:
        raise MarlinError(2, "marlin_workspace_bytes")
    return n


def new_workspace(max_M: int, K: int, N: int, device="cuda"):
    """Allocates the workspace with torch and zeroes it once, as the C ABI requires."""
    torch = _torch()
    return torch.zeros(workspace_bytes(max_M, K, N), dtype=torch.uint8, device=device)


def quantize_rtn(W, group_size: int, n_grid: int = 20, n_candidates: int = 10, stream=None):
    """marlin_quantize_rtn: fp16 weights [K, N] -> (q_kpacked int32 [K/8, N], scales fp16 [K/G, N]), the inputs of pack.

    Round to nearest with a per-group search over n_candidates clipping thresholds 1 - t / n_grid."""
    torch = _torch()
    W = _dev(W, torch.float16, "W")
    if W.dim() != 2:
        raise ValueError("W must be [K, N]")
    K, N = W.shape
    L = lib()
    sb = L.marlin_packed_scale_bytes(K, N, group_size)
    if L.marlin_packed_weight_bytes(K, N, 0) == 0:
        raise MarlinError(2, "marlin_quantize_rtn")
    if sb == 0:
        raise MarlinError(3, "marlin_quantize_rtn")
    q = torch.empty((K // 8, N), dtype=torch.int32, device=W.device)
    s = torch.empty((sb // (2 * N), N), dtype=torch.float16, device=W.device)
    _check(L.marlin_quantize_rtn(W.data_ptr(), q.data_ptr(), s.data_ptr(), K, N, group_size, n_grid, n_candidates,
                                 _stream_ptr(stream)), "marlin_quantize_rtn")
    return q, s


def pack(q_kpacked, scales, group_size: int, stream=None):
    """marlin_pack: canonical codes uint32(int32) [K/8, N] + fp16 scales [K/G, N] -> (w_packed, s_packed)."""
    torch = _torch()
    q = _dev(q_kpacked, torch.int32, "q_kpacked")
    s = _dev(scales, torch.float16, "scales")
    K, N = q.shape[0] * 8, q.shape[1]
    L = lib()
    wb, sb = L.marlin_packed_weight_bytes(K, N, 0), L.marlin_packed_scale_bytes(K, N, group_size)
    if wb == 0:
        raise MarlinError(2, "marlin_pack")
    if sb == 0:
        raise MarlinError(3, "marlin_pack")
    if s.numel() * 2 != sb:
        raise ValueError(f"scales has {s.numel()} elements, expected {sb // 2}")
    w_packed = torch.empty(wb, dtype=torch.uint8, device=q.device)
    s_packed = torch.empty(sb, dtype=torch.uint8, device=q.device)
    _check(L.marlin_pack(q.data_ptr(), s.data_ptr(), w_packed.data_ptr(), s_packed.data_ptr(), K, N, group_size,
                         _stream_ptr(stream)), "marlin_pack")
    return w_packed, s_packed


def unpack(w_packed, s_packed, K: int, N: int, group_size: int, stream=None):
    """marlin_unpack: the inverse of pack; returns (q_kpacked int32 [K/8, N], scales fp16 [K/G, N])."""
    torch = _torch()
    w = _dev(w_packed, torch.uint8, "w_packed")
    s = _dev(s_packed, torch.uint8, "s_packed")
    L = lib()
    sb = L.marlin_packed_scale_bytes(K, N, group_size)
    if w.numel() != L.marlin_packed_weight_bytes(K, N, 0) or s.numel() != sb or sb == 0:
        raise ValueError("packed buffer sizes do not match K, N, group_size")
    q = torch.empty((K // 8, N), dtype=torch.int32, device=w.device)
    sc = torch.empty((sb // 2 // N, N), dtype=torch.float16, device=w.device)
    _check(L.marlin_unpack(w.data_ptr(), s.data_ptr(), q.data_ptr(), sc.data_ptr(), K, N, group_size,
                           _stream_ptr(stream)), "marlin_unpack")
    return q, sc


def gemm(A, w_packed, s_packed, K: int, N: int, group_size: int, workspace, out=None, stream=None):
    """marlin_gemm: C[M, N] = A[M, K] . dequant(W).  `workspace` from new_workspace(max_M >= M, K, N)."""
    torch = _torch()
    A = _dev(A, torch.float16, "A")
    if A.dim() != 2 or A.shape[1] != K:
        raise ValueError("A must be [M, K]")
    M = A.shape[0]
    w = _dev(w_packed, torch.uint8, "w_packed")
    s = _dev(s_packed, torch.uint8, "s_packed")
    ws = _dev(workspace, torch.uint8, "workspace")
    L = lib()
    if w.numel() != L.marlin_packed_weight_bytes(K, N, 0) or s.numel() != L.marlin_packed_scale_bytes(K, N, group_size):
        raise ValueError("packed buffer sizes do not match K, N, group_size")
    if out is None:
        out = torch.empty((M, N), dtype=torch.float16, device=A.device)
    else:
        _dev(out, torch.float16, "out")
        if tuple(out.shape) != (M, N):
            raise ValueError("out must be [M, N]")
    _check(L.marlin_gemm(A.data_ptr(), w.data_ptr(), s.data_ptr(), out.data_ptr(), M, K, N, group_size,
                         ws.data_ptr(), ws.numel(), _stream_ptr(stream)), "marlin_gemm")
    return out


def pack_zeros(zeros, K: int, N: int, group_size: int, stream=None):
    """marlin_pack_zeros: zero points uint8 [K/G, N] (0..15) -> z_packed for gemm_zp."""
    torch = _torch()
    z = _dev(zeros, torch.uint8, "zeros")
    L = lib()
    sb = L.marlin_packed_scale_bytes(K, N, group_size)
    if sb == 0 or z.numel() * 2 != sb:
        raise ValueError("zeros must be [K/G, N] for a supported K, N, group_size")
    z_packed = torch.empty(sb, dtype=torch.uint8, device=z.device)
    _check(L.marlin_pack_zeros(z.data_ptr(), z_packed.data_ptr(), K, N, group_size, _stream_ptr(stream)), "marlin_pack_zeros")
    return z_packed


def unpack_zeros(z_packed, K: int, N: int, group_size: int, stream=None):
    """marlin_unpack_zeros: the inverse of pack_zeros; returns uint8 [K/G, N]."""
    torch = _torch()
    zq = _dev(z_packed, torch.uint8, "z_packed")
    L = lib()
    sb = L.marlin_packed_scale_bytes(K, N, group_size)
    if sb == 0 or zq.numel() != sb:
        raise ValueError("z_packed does not match K, N, group_size")
    z = torch.empty((sb // (2 * N), N), dtype=torch.uint8, device=zq.device)
    _check(L.marlin_unpack_zeros(zq.data_ptr(), z.data_ptr(), K, N, group_size, _stream_ptr(stream)), "marlin_unpack_zeros")
    return z


def gemm_zp(A, w_packed, s_packed, z_packed, K: int, N: int, group_size: int, workspace, out=None, stream=None):
    """marlin_gemm_zp: C = A . ((q - z) * s) with per-group zero points; N % 256 == 0."""
    torch = _torch()
    A = _dev(A, torch.float16, "A")
    if A.dim() != 2 or A.shape[1] != K:
        raise ValueError("A must be [M, K]")
    M = A.shape[0]
    w = _dev(w_packed, torch.uint8, "w_packed")
    s = _dev(s_packed, torch.uint8, "s_packed")
    z = _dev(z_packed, torch.uint8, "z_packed")
    ws = _dev(workspace, torch.uint8, "workspace")
    L = lib()
    sb = L.marlin_packed_scale_bytes(K, N, group_size)
    if w.numel() != L.marlin_packed_weight_bytes(K, N, 0) or s.numel() != sb or z.numel() != sb:
        raise ValueError("packed buffer sizes do not match K, N, group_size")
    if out is None:
        out = torch.empty((M, N), dtype=torch.float16, device=A.device)
    else:
        _dev(out, torch.float16, "out")
        if tuple(out.shape) != (M, N):
            raise ValueError("out must be [M, N]")
    _check(L.marlin_gemm_zp(A.data_ptr(), w.data_ptr(), s.data_ptr(), z.data_ptr(), out.data_ptr(), M, K, N, group_size,
                            ws.data_ptr(), ws.numel(), _stream_ptr(stream)), "marlin_gemm_zp")
    return out


def interleave_gate_up(q_gate, s_gate, q_up, s_up, group_size: int, stream=None):
    """marlin_interleave_gate_up: canonical (codes, scales) of the gate and up projections [K, I] each -> those of the
    fused layer [K, 2 I] in blocks of 16 columns (8 gate, 8 up)."""
    torch = _torch()
    qg, qu = _dev(q_gate, torch.int32, "q_gate"), _dev(q_up, torch.int32, "q_up")
    sg, su = _dev(s_gate, torch.float16, "s_gate"), _dev(s_up, torch.float16, "s_up")
    if qg.shape != qu.shape or sg.shape != su.shape or qg.shape[1] != sg.shape[1]:
        raise ValueError("gate and up must have the same shapes")
    K, I = qg.shape[0] * 8, qg.shape[1]
    q = torch.empty((K // 8, 2 * I), dtype=torch.int32, device=qg.device)
    s = torch.empty((sg.shape[0], 2 * I), dtype=torch.float16, device=qg.device)
    _check(lib().marlin_interleave_gate_up(qg.data_ptr(), sg.data_ptr(), qu.data_ptr(), su.data_ptr(), q.data_ptr(),
                                           s.data_ptr(), K, I, group_size, _stream_ptr(stream)), "marlin_interleave_gate_up")
    return q, s


def gemm_swiglu(A, w_packed, s_packed, K: int, N: int, group_size: int, workspace, out=None, stream=None):
    """marlin_gemm_swiglu: H[M, N/2] = silu(gate) * up of the fused gate_up layer (see interleave_gate_up)."""
    torch = _torch()
    A = _dev(A, torch.float16, "A")
    if A.dim() != 2 or A.shape[1] != K:
        raise ValueError("A must be [M, K]")
    M = A.shape[0]
    w = _dev(w_packed, torch.uint8, "w_packed")
    s = _dev(s_packed, torch.uint8, "s_packed")
    ws = _dev(workspace, torch.uint8, "workspace")
    L = lib()
    if w.numel() != L.marlin_packed_weight_bytes(K, N, 0) or s.numel() != L.marlin_packed_scale_bytes(K, N, group_size):
        raise ValueError("packed buffer sizes do not match K, N, group_size")
    if out is None:
        out = torch.empty((M, N // 2), dtype=torch.float16, device=A.device)
    else:
        _dev(out, torch.float16, "out")
        if tuple(out.shape) != (M, N // 2):
            raise ValueError("out must be [M, N / 2]")
    _check(L.marlin_gemm_swiglu(A.data_ptr(), w.data_ptr(), s.data_ptr(), out.data_ptr(), M, K, N, group_size,
                                ws.data_ptr(), ws.numel(), _stream_ptr(stream)), "marlin_gemm_swiglu")
    return out


def mlp_swiglu(A, w_gate_up, s_gate_up, w_down, s_down, K: int, I: int, N: int, group_size: int, workspace, H=None, out=None,
               stream=None):
    """marlin_mlp_swiglu: (silu(A . W_gate) * (A . W_up)) . W_down as two launches; returns C [M, N]."""
    torch = _torch()
    A = _dev(A, torch.float16, "A")
    if A.dim() != 2 or A.shape[1] != K:
        raise ValueError("A must be [M, K]")
    M = A.shape[0]
    ws = _dev(workspace, torch.uint8, "workspace")
    L = lib()
    wg, sg = _dev(w_gate_up, torch.uint8, "w_gate_up"), _dev(s_gate_up, torch.uint8, "s_gate_up")
    wd, sd = _dev(w_down, torch.uint8, "w_down"), _dev(s_down, torch.uint8, "s_down")
    if (wg.numel() != L.marlin_packed_weight_bytes(K, 2 * I, 0) or sg.numel() != L.marlin_packed_scale_bytes(K, 2 * I, group_size)
            or wd.numel() != L.marlin_packed_weight_bytes(I, N, 0) or sd.numel() != L.marlin_packed_scale_bytes(I, N, group_size)):
        raise ValueError("packed buffer sizes do not match K, I, N, group_size")
    if H is None:
        H = torch.empty((M, I), dtype=torch.float16, device=A.device)
    if out is None:
        out = torch.empty((M, N), dtype=torch.float16, device=A.device)
    _dev(H, torch.float16, "H")
    _dev(out, torch.float16, "out")
    if tuple(H.shape) != (M, I) or tuple(out.shape) != (M, N):
        raise ValueError("H must be [M, I] and out [M, N]")
    _check(L.marlin_mlp_swiglu(A.data_ptr(), wg.data_ptr(), sg.data_ptr(), wd.data_ptr(), sd.data_ptr(), H.data_ptr(),
                               out.data_ptr(), M, K, I, N, group_size, ws.data_ptr(), ws.numel(), _stream_ptr(stream)),
           "marlin_mlp_swiglu")
    return out


def pack_w8(q8, scales, group_size: int, stream=None):
    """marlin_pack_w8: 8-bit codes uint8 [K, N] + fp16 scales [K/G, N] -> (w_packed, s_packed); N % 256 == 0."""
    torch = _torch()
    q = _dev(q8, torch.uint8, "q8")
    s = _dev(scales, torch.float16, "scales")
    K, N = q.shape
    L = lib()
    wb, sb = L.marlin_packed_weight_bytes_w8(K, N), L.marlin_packed_scale_bytes(K, N, group_size)
    if wb == 0:
        raise MarlinError(2, "marlin_pack_w8")
    if sb == 0:
        raise MarlinError(3, "marlin_pack_w8")
    if s.numel() * 2 != sb:
        raise ValueError(f"scales has {s.numel()} elements, expected {sb // 2}")
    w_packed = torch.empty(wb, dtype=torch.uint8, device=q.device)
    s_packed = torch.empty(sb, dtype=torch.uint8, device=q.device)
    _check(L.marlin_pack_w8(q.data_ptr(), s.data_ptr(), w_packed.data_ptr(), s_packed.data_ptr(), K, N, group_size,
                            _stream_ptr(stream)), "marlin_pack_w8")
    return w_packed, s_packed


def unpack_w8(w_packed, s_packed, K: int, N: int, group_size: int, stream=None):
    """marlin_unpack_w8: the inverse of pack_w8; returns (q8 uint8 [K, N], scales fp16 [K/G, N])."""
    torch = _torch()
    w = _dev(w_packed, torch.uint8, "w_packed")
    s = _dev(s_packed, torch.uint8, "s_packed")
    L = lib()
    sb = L.marlin_packed_scale_bytes(K, N, group_size)
    if w.numel() != L.marlin_packed_weight_bytes_w8(K, N) or s.numel() != sb or sb == 0:
        raise ValueError("packed buffer sizes do not match K, N, group_size")
    q = torch.empty((K, N), dtype=torch.uint8, device=w.device)
    sc = torch.empty((sb // (2 * N), N), dtype=torch.float16, device=w.device)
    _check(L.marlin_unpack_w8(w.data_ptr(), s.data_ptr(), q.data_ptr(), sc.data_ptr(), K, N, group_size, _stream_ptr(stream)),
           "marlin_unpack_w8")
    return q, sc


def gemm_w8(A, w_packed, s_packed, K: int, N: int, group_size: int, workspace, out=None, stream=None):
    """marlin_gemm_w8: C = A . ((q - 128) * s) for 8-bit codes."""
    torch = _torch()
    A = _dev(A, torch.float16, "A")
    if A.dim() != 2 or A.shape[1] != K:
        raise ValueError("A must be [M, K]")
    M = A.shape[0]
    w = _dev(w_packed, torch.uint8, "w_packed")
    s = _dev(s_packed, torch.uint8, "s_packed")
    ws = _dev(workspace, torch.uint8, "workspace")
    L = lib()
    if w.numel() != L.marlin_packed_weight_bytes_w8(K, N) or s.numel() != L.marlin_packed_scale_bytes(K, N, group_size):
        raise ValueError("packed buffer sizes do not match K, N, group_size")
    if out is None:
        out = torch.empty((M, N), dtype=torch.float16, device=A.device)
    else:
        _dev(out, torch.float16, "out")
        if tuple(out.shape) != (M, N):
            raise ValueError("out must be [M, N]")
    _check(L.marlin_gemm_w8(A.data_ptr(), w.data_ptr(), s.data_ptr(), out.data_ptr(), M, K, N, group_size,
                            ws.data_ptr(), ws.numel(), _stream_ptr(stream)), "marlin_gemm_w8")
    return out


def gemm_static_ws(A, w_packed, s_packed, K: int, N: int, group_size: int, out=None, stream=None):
    """marlin_gemm_static_ws: the layer for callers that cannot allocate or pass a workspace.

    Same result as `gemm`, M <= STATIC_WS_MAX_M only.  The scratch memory is a fixed array inside the
    library; calls on one device share it, so do not let two of them overlap on the GPU.  `out` should
    be supplied by callers that must not allocate (without it this binding asks torch for the output).
    """
    torch = _torch()
    A = _dev(A, torch.float16, "A")
    if A.dim() != 2 or A.shape[1] != K:
        raise ValueError("A must be [M, K]")
    M = A.shape[0]
    w = _dev(w_packed, torch.uint8, "w_packed")
    s = _dev(s_packed, torch.uint8, "s_packed")
    L = lib()
    if w.numel() != L.marlin_packed_weight_bytes(K, N, 0) or s.numel() != L.marlin_packed_scale_bytes(K, N, group_size):
        raise ValueError("packed buffer sizes do not match K, N, group_size")
    if out is None:
        out = torch.empty((M, N), dtype=torch.float16, device=A.device)
    else:
        _dev(out, torch.float16, "out")
        if tuple(out.shape) != (M, N):
            raise ValueError("out must be [M, N]")
    _check(L.marlin_gemm_static_ws(A.data_ptr(), w.data_ptr(), s.data_ptr(), out.data_ptr(), M, K, N, group_size,
                                   _stream_ptr(stream)), "marlin_gemm_static_ws")
    return out


def pack_sparse24(qc_kpacked, idx, scales, group_size: int, stream=None):
    """marlin_pack_sparse24: kept codes int32 [K/16, N], positions uint8 [K/2, N], scales fp16 [K/G, N]."""
    torch = _torch()
    qc = _dev(qc_kpacked, torch.int32, "qc_kpacked")
    ix = _dev(idx, torch.uint8, "idx")
    s = _dev(scales, torch.float16, "scales")
    K, N = qc.shape[0] * 16, qc.shape[1]
    if tuple(ix.shape) != (K // 2, N):
        raise ValueError("idx must be [K/2, N]")
    L = lib()
    wb, mb, sb = (L.marlin_packed_weight_bytes(K, N, 1), L.marlin_packed_meta_bytes(K, N),
                  L.marlin_packed_scale_bytes(K, N, group_size))
    if wb == 0 or mb == 0:
        raise MarlinError(2, "marlin_pack_sparse24")
    if sb == 0:
        raise MarlinError(3, "marlin_pack_sparse24")
    w_packed = torch.empty(wb, dtype=torch.uint8, device=qc.device)
    m_packed = torch.empty(mb, dtype=torch.uint8, device=qc.device)
    s_packed = torch.empty(sb, dtype=torch.uint8, device=qc.device)
    _check(L.marlin_pack_sparse24(qc.data_ptr(), ix.data_ptr(), s.data_ptr(), w_packed.data_ptr(),
                                  m_packed.data_ptr(), s_packed.data_ptr(), K, N, group_size, _stream_ptr(stream)),
           "marlin_pack_sparse24")
    return w_packed, m_packed, s_packed


def unpack_sparse24(w_packed, meta_packed, s_packed, K: int, N: int, group_size: int, stream=None):
    torch = _torch()
    w = _dev(w_packed, torch.uint8, "w_packed")
    m = _dev(meta_packed, torch.uint8, "meta_packed")
    s = _dev(s_packed, torch.uint8, "s_packed")
    L = lib()
    sb = L.marlin_packed_scale_bytes(K, N, group_size)
    qc = torch.empty((K // 16, N), dtype=torch.int32, device=w.device)
    ix = torch.empty((K // 2, N), dtype=torch.uint8, device=w.device)
    sc = torch.empty((sb // 2 // N, N), dtype=torch.float16, device=w.device)
    _check(L.marlin_unpack_sparse24(w.data_ptr(), m.data_ptr(), s.data_ptr(), qc.data_ptr(), ix.data_ptr(),
                                    sc.data_ptr(), K, N, group_size, _stream_ptr(stream)), "marlin_unpack_sparse24")
    return qc, ix, sc


def gemm_sparse24(A, w_packed, meta_packed, s_packed, K: int, N: int, group_size: int, workspace, out=None,
                  stream=None):
    torch = _torch()
    A = _dev(A, torch.float16, "A")
    if A.dim() != 2 or A.shape[1] != K:
        raise ValueError("A must be [M, K]")
    M = A.shape[0]
    w = _dev(w_packed, torch.uint8, "w_packed")
    m = _dev(meta_packed, torch.uint8, "meta_packed")
    s = _dev(s_packed, torch.uint8, "s_packed")
    ws = _dev(workspace, torch.uint8, "workspace")
    if out is None:
        out = torch.empty((M, N), dtype=torch.float16, device=A.device)
    _check(lib().marlin_gemm_sparse24(A.data_ptr(), w.data_ptr(), m.data_ptr(), s.data_ptr(), out.data_ptr(), M, K,
                                      N, group_size, ws.data_ptr(), ws.numel(), _stream_ptr(stream)),
           "marlin_gemm_sparse24")
    return out


class Layer:
    """A packed layer bound to its workspace: its buffers are checked once, here, so that a call only checks A,
    reads three pointers and makes the one foreign call (marlin_gemm, marlin_gemm_sparse24, marlin_gemm_zp or
    marlin_gemm_w8 by what the layer has).  Argument marshalling only, like the functions above.

        layer = Layer(w_packed, s_packed, K, N, group_size, workspace)      # dense 4-bit
        layer = Layer(..., meta_packed=meta)                                # 2:4
        layer = Layer(..., z_packed=z)                                      # zero points
        layer = Layer(..., w8=True)                                         # 8-bit codes
        C = layer(A)            # or layer(A, out=C, stream=s)
    """

    def __init__(self, w_packed, s_packed, K: int, N: int, group_size: int, workspace, meta_packed=None, z_packed=None,
                 w8: bool = False, max_M: Optional[int] = None):
        torch = _torch()
        L = lib()
        if sum(x is not None for x in (meta_packed, z_packed)) + (1 if w8 else 0) > 1:
            raise ValueError("a layer is one of: dense, 2:4 (meta_packed), zero points (z_packed), 8-bit (w8)")
        self.K, self.N, self.G = int(K), int(N), int(group_size)
        w = _dev(w_packed, torch.uint8, "w_packed")
        sc = _dev(s_packed, torch.uint8, "s_packed")
        ws = _dev(workspace, torch.uint8, "workspace")
        wbytes = L.marlin_packed_weight_bytes_w8(K, N) if w8 else L.marlin_packed_weight_bytes(K, N, 1 if meta_packed is not None else 0)
        sbytes = L.marlin_packed_scale_bytes(K, N, group_size)
        if wbytes == 0 or sbytes == 0 or w.numel() != wbytes or sc.numel() != sbytes:
            raise ValueError("packed buffer sizes do not match K, N, group_size")
        self._keep = [w, sc, ws]
        extra = None
        if meta_packed is not None:
            extra = _dev(meta_packed, torch.uint8, "meta_packed")
            if extra.numel() != L.marlin_packed_meta_bytes(K, N):
                raise ValueError("meta_packed does not match K, N")
            self._fn, self._what = L.marlin_gemm_sparse24, "marlin_gemm_sparse24"
        elif z_packed is not None:
            extra = _dev(z_packed, torch.uint8, "z_packed")
            if extra.numel() != sbytes:
                raise ValueError("z_packed does not match K, N, group_size")
            self._fn, self._what = L.marlin_gemm_zp, "marlin_gemm_zp"
        elif w8:
            self._fn, self._what = L.marlin_gemm_w8, "marlin_gemm_w8"
        else:
            self._fn, self._what = L.marlin_gemm, "marlin_gemm"
        if extra is not None:
            self._keep.append(extra)
        self._kind = 1 if meta_packed is not None else (2 if z_packed is not None else 0)
        self._w, self._s, self._x = w.data_ptr(), sc.data_ptr(), (extra.data_ptr() if extra is not None else 0)
        self._ws, self._ws_bytes = ws.data_ptr(), ws.numel()
        self._device = w.device
        self._f16 = torch.float16
        self._empty = torch.empty
        self._current_stream = torch.cuda.current_stream
        if max_M is not None and self._ws_bytes < L.marlin_workspace_bytes(max_M, K, N):
            raise ValueError("workspace smaller than marlin_workspace_bytes(max_M, K, N)")

    def __call__(self, A, out=None, stream=None):
        if A.dtype != self._f16 or not A.is_cuda or not A.is_contiguous() or A.dim() != 2 or A.shape[1] != self.K:
            raise ValueError("A must be a contiguous fp16 CUDA tensor [M, K]")
        M = A.shape[0]
        if out is None:
            out = self._empty((M, self.N), dtype=self._f16, device=self._device)
        elif out.dtype != self._f16 or not out.is_cuda or not out.is_contiguous() or tuple(out.shape) != (M, self.N):
            raise ValueError("out must be a contiguous fp16 CUDA tensor [M, N]")
        sp = (stream if stream is not None else self._current_stream()).cuda_stream
        k = self._kind
        if k == 0:
            st = self._fn(A.data_ptr(), self._w, self._s, out.data_ptr(), M, self.K, self.N, self.G, self._ws, self._ws_bytes, sp)
        elif k == 1:
            st = self._fn(A.data_ptr(), self._w, self._x, self._s, out.data_ptr(), M, self.K, self.N, self.G, self._ws,
                          self._ws_bytes, sp)
        else:
            st = self._fn(A.data_ptr(), self._w, self._s, self._x, out.data_ptr(), M, self.K, self.N, self.G, self._ws,
                          self._ws_bytes, sp)
        if st != 0:
            raise MarlinError(st, self._what)
        return out

    def prepare(self, A, out=None, stream=None):
        """Checks A and out once and returns a function of no arguments that makes the foreign call on exactly these
        buffers and this stream and returns `out`: for callers that reuse fixed device buffers step after step."""
        if A.dtype != self._f16 or not A.is_cuda or not A.is_contiguous() or A.dim() != 2 or A.shape[1] != self.K:
            raise ValueError("A must be a contiguous fp16 CUDA tensor [M, K]")
        M = A.shape[0]
        if out is None:
            out = self._empty((M, self.N), dtype=self._f16, device=self._device)
        elif out.dtype != self._f16 or not out.is_cuda or not out.is_contiguous() or tuple(out.shape) != (M, self.N):
            raise ValueError("out must be a contiguous fp16 CUDA tensor [M, N]")
        sp = (stream if stream is not None else self._current_stream()).cuda_stream
        head = (A.data_ptr(), self._w)
        mid = (self._s,) if self._kind == 0 else ((self._x, self._s) if self._kind == 1 else (self._s, self._x))
        args = head + mid + (out.data_ptr(), M, self.K, self.N, self.G, self._ws, self._ws_bytes, sp)
        fn, what, keep = self._fn, self._what, (A, out, stream, self)

        def call():
            st = fn(*args)
            if st != 0:
                raise MarlinError(st, what)
            return keep[1]
        return call


def read_status(workspace, stream=None) -> int:
    """marlin_read_status: synchronises the stream and returns the device-side status word."""
    torch = _torch()
    ws = _dev(workspace, torch.uint8, "workspace")
    return int(lib().marlin_read_status(ws.data_ptr(), _stream_ptr(stream)))


def plan_stripes(M: int, K: int, N: int, sm_count: int) -> Tuple[int, int, list]:
    """marlin_plan_stripes (host only): returns (n_tile, workers, bounds[workers + 1])."""
    L = lib()
    cap = 1024
    n_tile, workers = ctypes.c_int(0), ctypes.c_int(0)
    bounds = (ctypes.c_int64 * cap)()
    _check(L.marlin_plan_stripes(M, K, N, sm_count, ctypes.byref(n_tile), ctypes.byref(workers), bounds, cap),
           "marlin_plan_stripes")
    return n_tile.value, workers.value, list(bounds[: workers.value + 1])
