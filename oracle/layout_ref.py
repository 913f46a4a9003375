"""CPU restatement of the device weight layout -- TEST INFRASTRUCTURE ONLY.

Written from the written description of the packed layout (the design notes of this repository), not from the CUDA source;
used only to compare bytes with what ``marlin_pack`` writes on the GPU.  Nothing in the product
imports this file.

Dense layout: the packed buffer is a sequence of 4096-byte chunks, one per (k-block kb = k/128,
64-column block nb = n/64), ordered by super-columns of four chunks:
    chunk index = (nb/4) * 4 * (K/128) + kb * cs + nb % 4,   cs = min(4, N/64 - 4*(nb/4))
Inside a chunk, 16-byte vector v = (2*j + b)*32 + 4*g + slot holds 32 codes of column
    n = 64*nb + 16*j + 8*b + g,   slot = (c + g/2) % 4 for c = 0..3;
its word w = 2*h + u holds rows k = 128*kb + 64*h + 16*c + 8*u + o (o = 0..7), row offset o sitting in
nibble (o >> 1) + 4*(o & 1) (bits 4p..4p+3 for nibble p).
Scales: inside every run of 64 columns, packed position 8*g + 2*j + b holds column 16*j + 8*b + g; groups of 64 or
32 rows are regrouped per k-block and 256-column tile (see pack_scales).
"""
from __future__ import annotations

import numpy as np


def pack_dense_weights(Q: np.ndarray) -> np.ndarray:
    """Codes Q[K, N] (uint8, 0..15) -> packed uint32 words (1-D, K*N/8)."""
    K, N = Q.shape
    assert K % 128 == 0 and N % 64 == 0
    kb, nb, j, b, g, slot, h, u, p = np.meshgrid(
        np.arange(K // 128), np.arange(N // 64), np.arange(4), np.arange(2), np.arange(8), np.arange(4),
        np.arange(2), np.arange(2), np.arange(8), indexing="ij")
    c = (slot - g // 2) % 4     # the rows 16c.. of a column sit in slot (c + g/2) % 4
    o = 2 * (p & 3) + (p >> 2)  # row offset stored in nibble p
    n = 64 * nb + 16 * j + 8 * b + g
    k = 128 * kb + 64 * h + 16 * c + 8 * u + o
    codes = Q[k, n].astype(np.uint32)  # [kb, nb, j, b, g, slot, h, u, p]: already in word order inside a chunk
    words = np.zeros(codes.shape[:-1], dtype=np.uint32)
    for pp in range(8):
        words |= codes[..., pp] << np.uint32(4 * pp)
    chunks = words.reshape(K // 128, N // 64, 1024)  # [kb, nb, words of the chunk]
    KB, NB = K // 128, N // 64
    out = np.empty((KB * NB, 1024), dtype=np.uint32)
    for nb_ in range(NB):
        sc = nb_ // 4
        cs = min(4, NB - 4 * sc)
        idx = sc * 4 * KB + np.arange(KB) * cs + nb_ % 4
        out[idx] = chunks[:, nb_, :]
    return out.reshape(-1)


def pack_scales(S: np.ndarray, sub: int = 1) -> np.ndarray:
    """Scales S[K/G, N] fp16 -> packed order (same number of elements).

    sub = 1 (groups of 128 rows and more): rows stay in place, inside every run of 64 columns packed position
    8g + 2j + b holds column 16j + 8b + g.  sub = 2, 4 (groups of 64, 32 rows; N a multiple of 256): the same
    permutation inside the runs, and the rows regrouped per k-block and 256-column tile: [K/128][N/256][sub][256].
    """
    R, N = S.shape
    assert N % 64 == 0
    pos = np.arange(64)
    g, j, b = pos >> 3, (pos >> 1) & 3, pos & 1
    src = 16 * j + 8 * b + g
    P = S.reshape(R, N // 64, 64)[:, :, src].reshape(R, N)
    if sub == 1:
        return P
    assert N % 256 == 0 and R % sub == 0
    return P.reshape(R // sub, sub, N // 256, 256).transpose(0, 2, 1, 3).reshape(R, N)


# ---- 2:4 variant ---------------------------------------------------------------------------------------
# Per chunk (128 rows of the original K = 64 kept rows, 64 columns; chunks ordered as in the dense layout):
#   codes (512 words): word (j*32 + lane)*4 + t, lane = 4g + c; nibble p (r = p % 4, e = p // 4) = kept value e of
#     column 64nb + 16j + g + 8(r & 1), MMA group gamma = c + 4(r >> 1) of step t, where MMA group gamma stands for
#     the actual group Gamma = 4(gamma % 2) + gamma // 2 of the step's eight groups of four original rows;
#     kept-value row T = 2*(32kb + 8t + Gamma) + e.
#   metadata (256 words): word ((j // 2)*32 + lane)*4 + (j % 2)*2 + w is supplied by lane (g, c) for step
#     t = c // 2 + 2w; nibble x = idx_first | idx_second << 2 for column 64nb + 16j + g + 8(x // 4), MMA group
#     4(c % 2) + x % 4.

def _chunk_order(KB, NB):
    order = np.empty((KB, NB), dtype=np.int64)
    for nb_ in range(NB):
        sc = nb_ // 4
        cs = min(4, NB - 4 * sc)
        order[:, nb_] = sc * 4 * KB + np.arange(KB) * cs + nb_ % 4
    return order


# Layers whose N is a multiple of 256 use the WIDE layout (read by the tcgen05 kernel).  Records in the order
# T * (K/128) + kb for the 256-column tile T and the k-block kb:
#   codes (2048 words): word ((c*256 + n)*4 + w) holds kept values e = 32c + 8w + o (o = 0..7) of column 256T + n, value o in
#     nibble (o >> 1) + 4(o & 1); kept value e of the k-block is kept row 64kb + e.
#   metadata (1024 words): word ((128t + L)*4 + i) with L = 16a + 8h + r: bits 0-15 describe column 256T + 128t + 16a + r,
#     bits 16-31 column 256T + 128t + 16a + 8 + r; the four 4-bit entries of each half are idx_first | idx_second << 2 of the
#     groups 8i + 4h + 0..3 of the k-block's 32 groups of four original rows.

def _wide_sparse_codes(Qc: np.ndarray, K: int) -> np.ndarray:
    N = Qc.shape[1]
    KB, NT = K // 128, N // 256
    T, kb, c, n, w, o = np.meshgrid(np.arange(NT), np.arange(KB), np.arange(2), np.arange(256), np.arange(4), np.arange(8),
                                    indexing="ij")
    codes = Qc[64 * kb + 32 * c + 8 * w + o, 256 * T + n].astype(np.uint32)
    words = np.zeros(codes.shape[:-1], dtype=np.uint32)
    for oo in range(8):
        words |= codes[..., oo] << np.uint32(4 * ((oo >> 1) + 4 * (oo & 1)))
    return words.reshape(-1)


def _wide_sparse_meta(idx: np.ndarray, K: int) -> np.ndarray:
    N = idx.shape[1]
    KB, NT = K // 128, N // 256
    T, kb, t, a, h, r, i, hw, gq = np.meshgrid(np.arange(NT), np.arange(KB), np.arange(2), np.arange(8), np.arange(2),
                                               np.arange(8), np.arange(4), np.arange(2), np.arange(4), indexing="ij")
    col = 256 * T + 128 * t + 16 * a + 8 * hw + r
    g2 = 2 * (32 * kb + 8 * i + 4 * h + gq)
    nib = idx[g2, col].astype(np.uint32) | (idx[g2 + 1, col].astype(np.uint32) << np.uint32(2))
    words = np.zeros(nib.shape[:-2], dtype=np.uint32)
    for hh in range(2):
        for gg in range(4):
            words |= nib[..., hh, gg] << np.uint32(16 * hh + 4 * gg)
    return words.reshape(-1)  # order [T, kb, t, a, h, r, i] = record, lane 16a + 8h + r of half t, step i


def pack_sparse_codes(Qc: np.ndarray, K: int) -> np.ndarray:
    """Kept codes Qc[K/2, N] (uint8) -> packed uint32 words (K*N/16)."""
    N = Qc.shape[1]
    if N % 256 == 0:
        return _wide_sparse_codes(Qc, K)
    KB, NB = K // 128, N // 64
    kb, nb, j, g, c, t, p = np.meshgrid(np.arange(KB), np.arange(NB), np.arange(4), np.arange(8), np.arange(4),
                                        np.arange(4), np.arange(8), indexing="ij")
    r, e = p & 3, p >> 2
    n = 64 * nb + 16 * j + g + 8 * (r & 1)
    gamma = c + 4 * (r >> 1)
    Gamma = 4 * (gamma % 2) + gamma // 2
    T = 2 * (32 * kb + 8 * t + Gamma) + e
    codes = Qc[T, n].astype(np.uint32)
    words = np.zeros(codes.shape[:-1], dtype=np.uint32)
    for pp in range(8):
        words |= codes[..., pp] << np.uint32(4 * pp)
    chunks = words.reshape(KB, NB, 512)
    out = np.empty((KB * NB, 512), dtype=np.uint32)
    out[_chunk_order(KB, NB).reshape(-1)] = chunks.reshape(KB * NB, 512)
    return out.reshape(-1)


def pack_sparse_meta(idx: np.ndarray, K: int) -> np.ndarray:
    """Positions idx[K/2, N] (uint8, 0..3) -> packed uint32 metadata words (K*N/32)."""
    N = idx.shape[1]
    if N % 256 == 0:
        return _wide_sparse_meta(idx, K)
    KB, NB = K // 128, N // 64
    kb, nb, jh, g, c, jl, w, x = np.meshgrid(np.arange(KB), np.arange(NB), np.arange(2), np.arange(8), np.arange(4),
                                             np.arange(2), np.arange(2), np.arange(8), indexing="ij")
    j = 2 * jh + jl
    t = c // 2 + 2 * w
    n = 64 * nb + 16 * j + g + 8 * (x >> 2)
    gamma = 4 * (c % 2) + (x & 3)
    Gamma = 4 * (gamma % 2) + gamma // 2
    G2 = 2 * (32 * kb + 8 * t + Gamma)
    nib = idx[G2, n].astype(np.uint32) | (idx[G2 + 1, n].astype(np.uint32) << np.uint32(2))
    words = np.zeros(nib.shape[:-1], dtype=np.uint32)
    for xx in range(8):
        words |= nib[..., xx] << np.uint32(4 * xx)
    chunks = words.reshape(KB, NB, 256)  # order inside: [jh, g, c, jl, w] = ((jh*32 + lane)*4 + jl*2 + w)
    out = np.empty((KB * NB, 256), dtype=np.uint32)
    out[_chunk_order(KB, NB).reshape(-1)] = chunks.reshape(KB * NB, 256)
    return out.reshape(-1)
