"""Layers with per-group zero points (marlin_pack_zeros, marlin_gemm_zp) against the CPU oracle (oracle/zp_ref.py),
through the C ABI.  Bound: |C - C_ref| <= 5e-3 * (|C_ref| + rms(C_ref)); integer closed forms bit for bit."""
import numpy as np
import pytest

from paper_2408_11743_b200 import inputs
from gpu_util import to_dev, to_host

pytestmark = pytest.mark.gpu

MODES = [{}, {"MARLIN_B200_TC_SPLIT": "0", "MARLIN_B200_SPLIT": "0"}, {"MARLIN_B200_TC_CLUSTER": "0", "MARLIN_B200_CLUSTER": "0"},
         {"MARLIN_B200_NW": "1"}, {"MARLIN_B200_NW": "4", "MARLIN_B200_SPLIT": "0"},
         {"MARLIN_B200_CW": "12"}, {"MARLIN_B200_CW": "12", "MARLIN_B200_NW": "2", "MARLIN_B200_SPLIT": "0"},
         {"MARLIN_B200_CW": "12", "MARLIN_B200_NW": "1", "MARLIN_B200_CLUSTER": "0"}]


@pytest.fixture(scope="module")
def marlin():
    import torch
    assert torch.cuda.is_available()
    import paper_2408_11743_b200 as m
    m.lib()
    return m


class ZpLayer:
    def __init__(self, marlin, q_kpacked, S, Z, G, max_M):
        self.m, self.K, self.N, self.G = marlin, q_kpacked.shape[0] * 8, q_kpacked.shape[1], G
        self.w, self.s = marlin.pack(to_dev(q_kpacked), to_dev(S), G)
        self.z = marlin.pack_zeros(to_dev(Z), self.K, self.N, G)
        self.ws = marlin.new_workspace(max_M, self.K, self.N)

    def __call__(self, A):
        import torch
        out = self.m.gemm_zp(to_dev(A), self.w, self.s, self.z, self.K, self.N, self.G, self.ws)
        torch.cuda.synchronize()
        assert self.m.read_status(self.ws) == 0
        return to_host(out)


def _case(M, K, N, G, seed):
    case = inputs.make_dense(M, K, N, G, seed=seed)
    rng = np.random.default_rng(seed + 1)
    Z = rng.integers(0, 16, size=case.S.shape, dtype=np.uint8)
    return case, Z


@pytest.mark.parametrize("K,N,G", [(256, 256, 128), (1024, 512, 64), (512, 768, 32), (1152, 256, 384), (512, 256, -1),
                                   (256, 64, 128), (512, 320, 128), (1024, 192, -1)])
def test_zero_point_pack_matches_the_layout_and_round_trips(marlin, K, N, G):
    import torch
    from oracle import layout_ref
    Gn = K if G == -1 else G
    rng = np.random.default_rng(K + N)
    Z = rng.integers(0, 16, size=(K // Gn, N), dtype=np.uint8)
    zq = marlin.pack_zeros(to_dev(Z), K, N, G)
    torch.cuda.synchronize()
    want = layout_ref.pack_scales(Z.astype(np.float16), sub=1 if Gn >= 128 else 128 // Gn)
    assert np.array_equal(to_host(zq).view(np.float16).reshape(want.shape), want)
    assert np.array_equal(to_host(marlin.unpack_zeros(zq, K, N, G)), Z)


@pytest.mark.parametrize("M,K,N,G", [(1, 1024, 256, 128), (16, 2048, 512, 128), (40, 1024, 768, 64), (64, 512, 256, 32),
                                     (128, 2048, 1024, 128), (100, 1152, 256, 384), (8, 1024, 512, -1), (300, 1024, 512, 128),
                                     (16, 8192, 8192, 128),
                                     # the warp-level kernel: up to 16 rows at any N, and in slabs of 16 rows where N is not a multiple of 256
                                     (1, 256, 64, 128), (5, 1024, 192, 128), (8, 4096, 320, 128), (9, 2048, 448, 256), (16, 1152, 128, 384),
                                     (16, 8192, 64, -1), (3, 28672, 128, -1), (40, 1024, 192, 128), (100, 512, 320, -1), (8, 4096, 4096, 128),
                                     (2, 11008, 4096, 128)])
def test_random_inputs_match_the_oracle(marlin, oracle_lib, M, K, N, G):
    from oracle import zp_ref
    case, Z = _case(M, K, N, G, seed=M + K + N)
    C = ZpLayer(marlin, case.q_kpacked, case.S, Z, G, M)(case.A)
    if K * N <= 1 << 21:
        ref = zp_ref.gemm_zp(case.A, case.q_kpacked, case.S, Z, case.G)
        bad, worst, rms = oracle_lib.check_tolerance(C, ref)
    else:
        # the full-size layer on sampled columns
        ns = np.random.default_rng(3).integers(0, N, 64)
        from oracle import unpack_q
        Q = unpack_q(case.q_kpacked)[:, ns]
        W = zp_ref.dequant_zp(Q, np.ascontiguousarray(case.S[:, ns]), np.ascontiguousarray(Z[:, ns]), case.G)
        ref = oracle_lib.f64_to_f16(case.A.astype(np.float64) @ W)
        bad, worst, rms = oracle_lib.check_tolerance(np.ascontiguousarray(C[:, ns]), ref)
    assert bad == 0, f"{bad} elements out of tolerance, worst ratio {worst:.3f}, rms {rms:.3f}"


@pytest.mark.parametrize("mode", range(len(MODES)))
@pytest.mark.parametrize("M,K,N,G", [(3, 1024, 256, 128), (33, 1024, 512, 64), (128, 2048, 256, -1), (200, 512, 512, 32),
                                     (8, 2048, 192, 128), (16, 4096, 512, 128), (12, 2048, 320, -1), (1, 8192, 1024, 256)])
def test_integer_closed_form_is_bit_exact(marlin, monkeypatch, mode, M, K, N, G):
    from oracle import zp_ref
    for k, v in MODES[mode].items():
        monkeypatch.setenv(k, v)
    rng = np.random.default_rng(M + K + N + mode)
    Gn = K if G == -1 else G
    Q = rng.integers(0, 16, size=(K, N), dtype=np.uint8)
    Z = rng.integers(0, 16, size=(K // Gn, N), dtype=np.uint8)
    A = rng.integers(-3, 4, size=(M, K)).astype(np.float16)
    S = np.ldexp(1.0, rng.integers(-4, 1, size=(K // Gn, N))).astype(np.float16)
    q = inputs.kpack(Q)
    C = ZpLayer(marlin, q, S, Z, G, M)(A)
    assert np.array_equal(C.view(np.uint16), zp_ref.gemm_zp(A, q, S, Z, Gn).view(np.uint16))


def test_unit_vectors_read_back_every_weight(marlin):
    # row m = unit vector of k = m: C[m, n] = (Q[m, n] - Z[m / G, n]) * S[m / G, n] exactly, for every zero point 0..15
    K, N, G = 128, 256, 32
    rng = np.random.default_rng(8)
    Q = rng.integers(0, 16, size=(K, N), dtype=np.uint8)
    Z = (np.arange(N)[None, :] + np.arange(K // G)[:, None]).astype(np.uint8) % 16
    expo = rng.integers(-5, 2, size=(K // G, N))
    S = np.ldexp(1.0, expo).astype(np.float16)
    A = np.eye(K, dtype=np.float16)
    C = ZpLayer(marlin, inputs.kpack(Q), S, Z, G, K)(A).astype(np.float64)
    want = (Q.astype(np.float64) - np.repeat(Z, G, axis=0)) * np.repeat(np.ldexp(1.0, expo), G, axis=0)
    assert np.array_equal(C, want)


def test_unit_vectors_through_the_warp_level_kernel(marlin):
    # 16 unit vectors at a time (the warp-level kernel), every zero point 0..15, N not a multiple of 256
    K, N, G = 256, 192, 128
    rng = np.random.default_rng(9)
    Q = rng.integers(0, 16, size=(K, N), dtype=np.uint8)
    Z = (np.arange(N)[None, :] + 5 * np.arange(K // G)[:, None]).astype(np.uint8) % 16
    expo = rng.integers(-5, 2, size=(K // G, N))
    S = np.ldexp(1.0, expo).astype(np.float16)
    layer = ZpLayer(marlin, inputs.kpack(Q), S, Z, G, 16)
    for k0 in range(0, K, 16):
        A = np.zeros((16, K), dtype=np.float16)
        A[np.arange(16), k0 + np.arange(16)] = 1.0
        want = (Q[k0:k0 + 16].astype(np.float64) - Z[k0 // G][None, :]) * np.ldexp(1.0, expo[k0 // G])[None, :]
        assert np.array_equal(layer(A).astype(np.float64), want), k0


def test_activations_with_offset_and_outliers(marlin, oracle_lib):
    # the zero-point term (8 - z) * sum_k a is large against the result when the activations have a mean: the bound
    # must still hold
    from oracle import zp_ref
    M, K, N, G = 8, 4096, 512, 128
    case, Z = _case(M, K, N, G, seed=4)
    A = (case.A.astype(np.float32) + 0.75).astype(np.float16)
    A[:, ::97] *= 40
    C = ZpLayer(marlin, case.q_kpacked, case.S, Z, G, M)(A)
    bad, worst, rms = oracle_lib.check_tolerance(C, zp_ref.gemm_zp(A, case.q_kpacked, case.S, Z, G))
    assert bad == 0, f"{bad} elements out of tolerance, worst ratio {worst:.3f}, rms {rms:.3f}"


def test_errors(marlin):
    import torch
    K, N, G = 256, 320, 64
    z = torch.zeros((K // G, N), dtype=torch.uint8, device="cuda")
    with pytest.raises((marlin.MarlinError, ValueError)):
        marlin.pack_zeros(z, K, N, G)  # groups of 64 rows need N to be a multiple of 256
