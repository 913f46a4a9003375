"""GPU parity of the tcgen05 kernel with deferred scales and 128-column tiles (gemm_tcd.cu) through the C ABI.

By default that kernel only takes batches above 16 rows on layers whose N is a multiple of 128 but not of 256;
MARLIN_B200_TCD=1 makes it take every batch size on every layer whose N is a multiple of 128, which is how
these tests reach all of its instances (16, 32 and 64 padded rows), pipelines longer than its stage ring,
stripes that cross column tiles, and both scale modes.

Bound: |C - C_ref| <= 5e-3 * (|C_ref| + rms(C_ref)) per element; integer-valued closed forms bit for bit.
"""
import numpy as np
import pytest

from paper_2408_11743_b200 import inputs
from gpu_util import DenseLayer, to_dev, to_host

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def marlin():
    import torch
    assert torch.cuda.is_available()
    import paper_2408_11743_b200 as m
    m.lib()
    return m


SHAPES = [
    (1, 128, 128, 128), (16, 256, 128, 128), (3, 512, 256, 128), (16, 1024, 512, 128), (8, 2048, 1536, -1),
    (13, 2048, 512, 256), (16, 4096, 4096, 128), (32, 2048, 1024, 128), (32, 4096, 4096, 128), (33, 1024, 512, 128),
    (64, 2048, 1024, 128), (64, 4096, 4096, -1), (5, 11008, 256, 128), (16, 28672, 1024, 128), (1, 8192, 8192, 128),
    (40, 1152, 512, 384), (24, 1152, 384, 384), (100, 1024, 640, -1), (150, 512, 384, 128), (17, 3072, 128, 128),
]


@pytest.mark.parametrize("M,K,N,G", SHAPES)
def test_tcd_kernel_matches_oracle_and_is_reproducible(marlin, oracle_lib, monkeypatch, M, K, N, G):
    monkeypatch.setenv("MARLIN_B200_TCD", "1")
    case = inputs.make_dense(M, K, N, G, seed=3000 + M + K + N)
    layer = DenseLayer(marlin, case.q_kpacked, case.S, G, max_M=M)
    C = layer(case.A)
    bad, worst, rms = oracle_lib.check_tolerance(C, oracle_lib.gemm(case.A, case.q_kpacked, case.S, case.G))
    assert bad == 0, f"{bad} elements out of tolerance, worst ratio {worst:.3f}, rms {rms:.3f}"
    # partial tiles are added in worker order by whoever arrives last: the same bits on every call
    for _ in range(3):
        assert np.array_equal(layer(case.A).view(np.uint16), C.view(np.uint16))
    assert np.all(to_host(layer.ws[256:8192]) == 0)  # arrival counters left clean


@pytest.mark.parametrize("M,K,N,G", [(2, 4096, 256, 128), (16, 8192, 512, 128), (33, 1024, 256, 128),
                                     (64, 2048, 512, 128), (48, 2048, 256, -1), (32, 4096, 1024, 256)])
def test_tcd_integer_closed_form_is_bit_exact(marlin, oracle_lib, monkeypatch, M, K, N, G):
    # scales powers of two, activations small integers: every partial sum is exact in fp32, also with the
    # offsets of the exponent trick riding along (|1032 * 3 * 128| < 2^24)
    monkeypatch.setenv("MARLIN_B200_TCD", "1")
    rng = np.random.default_rng(M + K)
    Q = rng.integers(0, 16, size=(K, N), dtype=np.uint8)
    A = rng.integers(-3, 4, size=(M, K)).astype(np.float16)
    Gn = K if G == -1 else G
    S = np.ldexp(1.0, rng.integers(-4, 1, size=(K // Gn, N))).astype(np.float16)
    q = inputs.kpack(Q)
    C = DenseLayer(marlin, q, S, G, max_M=M)(A)
    assert np.array_equal(C.view(np.uint16), oracle_lib.gemm(A, q, S, Gn).view(np.uint16))


@pytest.mark.parametrize("M", [16, 32, 64])
def test_tcd_one_hot_rows_probe_every_k_position(marlin, monkeypatch, M):
    monkeypatch.setenv("MARLIN_B200_TCD", "1")
    K, N, G = 512, 256, 128
    rng = np.random.default_rng(50 + M)
    Q = rng.integers(0, 16, size=(K, N), dtype=np.uint8)
    expo = rng.integers(-5, 2, size=(K // G, N))
    S = np.ldexp(1.0, expo).astype(np.float16)
    layer = DenseLayer(marlin, inputs.kpack(Q), S, G, max_M=M)
    for k0 in range(0, K, M):
        A = np.zeros((M, K), dtype=np.float16)
        A[np.arange(M), k0 + np.arange(M)] = 1.0
        want = np.stack([(Q[k0 + i].astype(np.float64) - 8) * np.ldexp(1.0, expo[(k0 + i) // G]) for i in range(M)])
        assert np.array_equal(layer(A).astype(np.float64), want), f"rows {k0}..{k0 + M - 1}"


def test_default_routing_uses_it_for_n_multiple_of_128_only(marlin, oracle_lib):
    # N = 384 (no 256-column tiles) at 40 rows: one launch of this kernel instead of three of the warp-level one
    case = inputs.make_dense(40, 2048, 384, 128, seed=8)
    C = DenseLayer(marlin, case.q_kpacked, case.S, 128, max_M=40)(case.A)
    bad, worst, _ = oracle_lib.check_tolerance(C, oracle_lib.gemm(case.A, case.q_kpacked, case.S, 128))
    assert bad == 0, worst


def test_tcd_long_stream_of_overlapping_launches_is_stable(marlin, monkeypatch):
    import torch
    monkeypatch.setenv("MARLIN_B200_TCD", "1")
    M, K, N = 16, 4096, 4096
    case0 = inputs.make_dense(M, K, N, 128, seed=5)
    case1 = inputs.make_dense(M, K, N, 128, seed=6)
    layer = DenseLayer(marlin, case0.q_kpacked, case0.S, 128, max_M=M)
    A = [to_dev(case0.A), to_dev(case1.A)]
    want = []
    for a in A:
        want.append(to_host(marlin.gemm(a, layer.w, layer.s, K, N, 128, layer.ws)).copy())
        torch.cuda.synchronize()
    C = [torch.empty((M, N), dtype=torch.float16, device="cuda") for _ in range(2)]
    for rep in range(3):
        for i in range(120):
            marlin.gemm(A[i % 2], layer.w, layer.s, K, N, 128, layer.ws, out=C[i % 2])
        torch.cuda.synchronize()
        assert marlin.read_status(layer.ws) == 0
        for i in range(2):
            assert np.array_equal(to_host(C[i]).view(np.uint16), want[i].view(np.uint16)), f"repetition {rep}, buffer {i}"
