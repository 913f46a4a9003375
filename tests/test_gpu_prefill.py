"""Batches above 128 rows: one launch whose stripes run over (column tile, slab of 128 rows, k-block), the layer
replicated in the unit numbering (Section 3.4, last paragraph; Section 5.1 "Large batch performance").

Compared with the CPU oracle through the C ABI: bit for bit on integer closed forms and unit-vector probes, within
|C - C_ref| <= 5e-3 * (|C_ref| + rms(C_ref)) on random inputs; in every partition and fix-up of the kernel.
"""
import numpy as np
import pytest

from paper_2408_11743_b200 import inputs
from gpu_util import DenseLayer, SparseLayer, to_dev, to_host

pytestmark = pytest.mark.gpu

MODES = [{}, {"MARLIN_B200_TC_SPLIT": "0"}, {"MARLIN_B200_TC_CLUSTER": "0"}]


@pytest.fixture(scope="module")
def marlin():
    import torch
    assert torch.cuda.is_available()
    import paper_2408_11743_b200 as m
    m.lib()
    return m


@pytest.mark.parametrize("mode", range(len(MODES)))
@pytest.mark.parametrize("M,K,N,G", [(129, 1024, 256, 128), (256, 2048, 512, 128), (300, 1024, 1024, -1),
                                     (512, 512, 256, 128), (1000, 1024, 768, 256), (2048, 256, 256, 128)])
def test_integer_closed_form_is_bit_exact_above_128_rows(marlin, oracle_lib, monkeypatch, mode, M, K, N, G):
    # powers of two as scales, small integers as activations: every partial sum is an exact fp32 value in any
    # order, so the result must equal the oracle bit for bit whichever CTAs shared a tile
    for k, v in MODES[mode].items():
        monkeypatch.setenv(k, v)
    rng = np.random.default_rng(3 * M + K + N)
    Q = rng.integers(0, 16, size=(K, N), dtype=np.uint8)
    A = rng.integers(-3, 4, size=(M, K)).astype(np.float16)
    Gn = K if G == -1 else G
    S = np.ldexp(1.0, rng.integers(-4, 1, size=(K // Gn, N))).astype(np.float16)
    q = inputs.kpack(Q)
    layer = DenseLayer(marlin, q, S, G, max_M=M)
    C = layer(A)
    C_ref = oracle_lib.gemm(A, q, S, Gn)
    assert np.array_equal(C.view(np.uint16), C_ref.view(np.uint16))
    # every row of every slab carries its own pattern: a slab written to the wrong rows would differ
    assert len({C[m].tobytes() for m in range(0, M, 7)}) == len(range(0, M, 7))
    ws = to_host(layer.ws)
    assert np.all(ws[256:] == 0)  # counters, partial slots and accumulation tiles are left clean


@pytest.mark.parametrize("mode", range(len(MODES)))
def test_unit_vectors_reach_every_slab_and_k_position(marlin, monkeypatch, mode):
    # row m is the unit vector of k = (37 m) mod K: C[m, n] = (Q[k, n] - 8) * S[k / G, n] exactly
    for k, v in MODES[mode].items():
        monkeypatch.setenv(k, v)
    K, N, G, M = 1024, 512, 128, 700
    rng = np.random.default_rng(5)
    Q = rng.integers(0, 16, size=(K, N), dtype=np.uint8)
    expo = rng.integers(-5, 2, size=(K // G, N))
    S = np.ldexp(1.0, expo).astype(np.float16)
    ks = (37 * np.arange(M)) % K
    A = np.zeros((M, K), dtype=np.float16)
    A[np.arange(M), ks] = 1.0
    C = DenseLayer(marlin, inputs.kpack(Q), S, G, max_M=M)(A).astype(np.float64)
    want = (Q[ks].astype(np.float64) - 8) * np.ldexp(1.0, expo[ks // G])
    assert np.array_equal(C, want)


@pytest.mark.parametrize("M,K,N,G", [(130, 2048, 1024, 128), (384, 4096, 512, 128), (1024, 1024, 2048, -1),
                                     (777, 2048, 256, 64), (260, 1024, 512, 32)])
def test_random_inputs_match_oracle_above_128_rows(marlin, oracle_lib, M, K, N, G):
    case = inputs.make_dense(M, K, N, G, seed=M + K)
    C = DenseLayer(marlin, case.q_kpacked, case.S, G, max_M=M)(case.A)
    bad, worst, rms = oracle_lib.check_tolerance(C, oracle_lib.gemm(case.A, case.q_kpacked, case.S, case.G))
    assert bad == 0, f"{bad} elements out of tolerance, worst ratio {worst:.3f}, rms {rms:.3f}"


def test_smaller_batches_reuse_a_large_workspace(marlin, oracle_lib):
    # one layer object (workspace sized for 600 rows) called with many batch sizes, large and small, in turn
    K, N, G = 1024, 512, 128
    case = inputs.make_dense(600, K, N, G, seed=77)
    layer = DenseLayer(marlin, case.q_kpacked, case.S, G, max_M=600)
    C_ref = oracle_lib.gemm(case.A, case.q_kpacked, case.S, G)
    fixed = marlin.workspace_bytes(1, 128, 64)  # a layer without accumulation tiles: counters and slot region alone
    for M in (600, 16, 129, 1, 128, 257, 64, 600):
        C = layer(case.A[:M])
        bad, worst, _ = oracle_lib.check_tolerance(C, np.ascontiguousarray(C_ref[:M]))
        assert bad == 0, (M, worst)
        ws = to_host(layer.ws)
        assert np.all(ws[256:8192] == 0)            # arrival counters
        assert np.all(ws[fixed:] == 0)              # accumulation tiles of the tcgen05 kernel (behind the slot region)


@pytest.mark.parametrize("M,K,N,G", [(200, 1024, 512, 128), (513, 2048, 256, -1)])
def test_sparse24_above_128_rows(marlin, oracle_lib, M, K, N, G):
    case = inputs.make_sparse24(M, K, N, G, seed=M)
    C = SparseLayer(marlin, case, M)(case.A)
    ref = oracle_lib.gemm_sparse24(case.A, case.qc_kpacked, case.idx, case.S, case.G)
    bad, worst, rms = oracle_lib.check_tolerance(C, ref)
    assert bad == 0, f"{bad} elements out of tolerance, worst ratio {worst:.3f}, rms {rms:.3f}"


def test_full_size_layer_at_1024_rows_on_sampled_outputs(marlin, oracle_lib):
    K, N, G, M = 8192, 8192, 128, 1024
    case = inputs.make_dense(M, K, N, G, seed=31)
    C = DenseLayer(marlin, case.q_kpacked, case.S, G, max_M=M)(case.A)
    rng = np.random.default_rng(4)
    ms = np.concatenate([rng.integers(0, M, 4000), np.arange(0, M, 11)])  # random samples and rows of every slab
    ns = np.concatenate([rng.integers(0, N, 4000), (97 * np.arange(0, M, 11)) % N])
    ref = oracle_lib.gemm_samples(case.A, case.q_kpacked, case.S, case.G, ms, ns)
    # the bound's rms is taken over the sampled outputs (a fair estimate of the full one)
    bad, worst, _ = oracle_lib.check_tolerance(np.ascontiguousarray(C[ms, ns]), ref)
    assert bad == 0, worst
    assert np.all(np.isfinite(C.astype(np.float32)))


@pytest.mark.parametrize("mode", range(len(MODES)))
@pytest.mark.parametrize("M,K,N,G", [(256, 2048, 512, 128), (384, 2048, 256, 128), (1000, 1024, 768, -1), (128, 2048, 512, 128),
                                     (40, 1024, 256, 128), (5000, 256, 512, 128)])
def test_nothing_is_written_outside_the_workspace(marlin, oracle_lib, monkeypatch, mode, M, K, N, G):
    # the workspace sits in the middle of a larger buffer filled with a pattern: every byte around it must survive
    # the call (the accumulation tiles of the fix-up are numbered per column tile, slab or worker, depending on the
    # partition; a wrong count or index would show here), and the call must still be correct
    import torch
    for k, v in MODES[mode].items():
        monkeypatch.setenv(k, v)
    case = inputs.make_dense(M, K, N, G, seed=5 * M + N)
    layer = DenseLayer(marlin, case.q_kpacked, case.S, G, max_M=M)
    need = layer.ws.numel()
    guard = 8 << 20
    big = torch.full((need + 2 * guard,), 0xA5, dtype=torch.uint8, device="cuda")
    big[guard:guard + need] = 0
    layer.ws = big[guard:guard + need]
    C = layer(case.A)
    bad, worst, _ = oracle_lib.check_tolerance(C, oracle_lib.gemm(case.A, case.q_kpacked, case.S, case.G))
    assert bad == 0, worst
    assert bool((big[:guard] == 0xA5).all()) and bool((big[guard + need:] == 0xA5).all())
    assert bool((big[guard + 256:guard + need] == 0).all())


def test_one_workspace_serves_layers_of_different_kinds_in_turn(marlin, oracle_lib, monkeypatch):
    # One buffer, sized as the largest of the calls' own requirements (each asked for at its own batch size), serves a
    # layer of the kernel with deferred scales (64 rows: partial-tile slots as wide as they get), a 2:4 layer and a
    # layer with groups of 64 rows on the tcgen05 kernel (accumulation tiles that must be zero at rest) and a layer
    # of the warp-level kernel forced onto the workspace fix-up, in turn on one stream without a synchronisation in
    # between.  The slots keep what a call left: they must never fall into another call's accumulation tiles.
    import torch
    monkeypatch.setenv("MARLIN_B200_CLUSTER", "0")
    d1 = inputs.make_dense(64, 2048, 2432, 128, seed=1)      # N not a multiple of 256: deferred scales, slots of every CTA
    sp = inputs.make_sparse24(16, 1024, 8192, 128, seed=2)   # 16 rows: 1 MB of accumulation tiles in the L2
    d3 = inputs.make_dense(8, 4096, 512, 128, seed=3)        # warp-level kernel, slots
    d4 = inputs.make_dense(24, 1024, 1024, 64, seed=4)       # groups of 64: tcgen05 kernel, accumulation tiles
    need = max(marlin.workspace_bytes(64, 2048, 2432), marlin.workspace_bytes(16, 1024, 8192),
               marlin.workspace_bytes(8, 4096, 512), marlin.workspace_bytes(24, 1024, 1024))
    ws = torch.zeros(need, dtype=torch.uint8, device="cuda")
    L1, L3, L4 = (DenseLayer(marlin, c.q_kpacked, c.S, c.G if c.G != c.K else -1, max_M=1) for c in (d1, d3, d4))
    L2 = SparseLayer(marlin, sp, 1)
    refs = {1: oracle_lib.gemm(d1.A, d1.q_kpacked, d1.S, d1.G), 3: oracle_lib.gemm(d3.A, d3.q_kpacked, d3.S, d3.G),
            4: oracle_lib.gemm(d4.A, d4.q_kpacked, d4.S, d4.G),
            2: oracle_lib.gemm_sparse24(sp.A, sp.qc_kpacked, sp.idx, sp.S, sp.G)}
    A = {1: to_dev(d1.A), 2: to_dev(sp.A), 3: to_dev(d3.A), 4: to_dev(d4.A)}
    outs = []
    for which in (1, 3, 2, 4, 1, 2, 3, 4, 2, 1):
        if which == 2:
            C = marlin.gemm_sparse24(A[2], L2.w, L2.meta, L2.s, L2.K, L2.N, L2.G, ws)
        else:
            L = {1: L1, 3: L3, 4: L4}[which]
            C = marlin.gemm(A[which], L.w, L.s, L.K, L.N, L.G, ws)
        outs.append((which, C))
    torch.cuda.synchronize()
    assert marlin.read_status(ws) == 0
    for i, (which, C) in enumerate(outs):
        bad, worst, _ = oracle_lib.check_tolerance(to_host(C), refs[which])
        assert bad == 0, (i, which, bad, worst)
    host = to_host(ws)
    assert np.all(host[256:8192] == 0)  # arrival counters
