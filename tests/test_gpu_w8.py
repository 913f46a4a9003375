"""8-bit weights (marlin_pack_w8, marlin_gemm_w8) against the CPU oracle (oracle/w8_ref.py), through the C ABI."""
import numpy as np
import pytest

from gpu_util import to_dev, to_host

pytestmark = pytest.mark.gpu

MODES = [{}, {"MARLIN_B200_TC_SPLIT": "0"}, {"MARLIN_B200_TC_CLUSTER": "0"}]


@pytest.fixture(scope="module")
def marlin():
    import torch
    assert torch.cuda.is_available()
    import paper_2408_11743_b200 as m
    m.lib()
    return m


class W8Layer:
    def __init__(self, marlin, Q8, S, G, max_M):
        self.m, self.K, self.N, self.G = marlin, Q8.shape[0], Q8.shape[1], G
        self.w, self.s = marlin.pack_w8(to_dev(Q8), to_dev(S), G)
        self.ws = marlin.new_workspace(max_M, self.K, self.N)

    def __call__(self, A):
        import torch
        out = self.m.gemm_w8(to_dev(A), self.w, self.s, self.K, self.N, self.G, self.ws)
        torch.cuda.synchronize()
        assert self.m.read_status(self.ws) == 0
        return to_host(out)


def _case(M, K, N, G, seed):
    rng = np.random.default_rng(seed)
    Gn = K if G == -1 else G
    Q8 = rng.integers(0, 256, size=(K, N), dtype=np.uint8)
    S = rng.uniform(0.0005, 0.002, size=(K // Gn, N)).astype(np.float16)
    A = rng.standard_normal((M, K)).astype(np.float16)
    return A, Q8, S, Gn


@pytest.mark.parametrize("K,N,G", [(256, 256, 128), (1024, 512, 64), (512, 768, -1)])
def test_pack_matches_the_layout_and_round_trips(marlin, K, N, G):
    import torch
    from oracle import layout_ref, w8_ref
    _, Q8, S, Gn = _case(1, K, N, G, K + N)
    w, s = marlin.pack_w8(to_dev(Q8), to_dev(S), G)
    torch.cuda.synchronize()
    assert np.array_equal(to_host(w), w8_ref.pack_w8(Q8))
    want_s = layout_ref.pack_scales(S, sub=1 if Gn >= 128 else 128 // Gn)
    assert np.array_equal(to_host(s).view(np.float16).reshape(want_s.shape), want_s)
    q2, s2 = marlin.unpack_w8(w, s, K, N, G)
    assert np.array_equal(to_host(q2), Q8) and np.array_equal(to_host(s2), S)


@pytest.mark.parametrize("M,K,N,G", [(1, 1024, 256, 128), (16, 2048, 512, 128), (40, 1024, 768, 64), (64, 512, 256, 32),
                                     (128, 2048, 1024, 128), (100, 1152, 256, 384), (8, 1024, 512, -1), (300, 1024, 512, 128),
                                     (16, 4096, 4096, 128)])
def test_random_inputs_match_the_oracle(marlin, oracle_lib, M, K, N, G):
    from oracle import w8_ref
    A, Q8, S, Gn = _case(M, K, N, G, M + K + N)
    C = W8Layer(marlin, Q8, S, G, M)(A)
    bad, worst, rms = oracle_lib.check_tolerance(C, w8_ref.gemm_w8(A, Q8, S, Gn))
    assert bad == 0, f"{bad} elements out of tolerance, worst ratio {worst:.3f}, rms {rms:.3f}"


@pytest.mark.parametrize("mode", range(len(MODES)))
@pytest.mark.parametrize("M,K,N,G", [(3, 1024, 256, 128), (33, 1024, 512, 64), (128, 1024, 256, -1), (200, 512, 512, 32)])
def test_integer_closed_form_is_bit_exact(marlin, monkeypatch, mode, M, K, N, G):
    # small integer activations, power-of-two scales: sums of integers below 2^24 in units of the scale, exact in any order
    from oracle import w8_ref
    for k, v in MODES[mode].items():
        monkeypatch.setenv(k, v)
    rng = np.random.default_rng(M + K + N + mode)
    Gn = K if G == -1 else G
    Q8 = rng.integers(0, 256, size=(K, N), dtype=np.uint8)
    A = rng.integers(-2, 3, size=(M, K)).astype(np.float16)
    S = np.ldexp(1.0, rng.integers(-8, -3, size=(K // Gn, N))).astype(np.float16)
    C = W8Layer(marlin, Q8, S, G, M)(A)
    assert np.array_equal(C.view(np.uint16), w8_ref.gemm_w8(A, Q8, S, Gn).view(np.uint16))


def test_unit_vectors_read_back_every_code(marlin):
    # every code 0..255 in every position of a k-block: C[m, n] = (Q8[m, n] - 128) * S exactly
    K, N, G = 256, 256, 128
    Q8 = ((np.arange(K)[:, None] * 7 + np.arange(N)[None, :] * 13) % 256).astype(np.uint8)
    expo = np.random.default_rng(1).integers(-9, -4, size=(K // G, N))
    S = np.ldexp(1.0, expo).astype(np.float16)
    layer = W8Layer(marlin, Q8, S, G, 128)
    for k0 in (0, 128):
        A = np.zeros((128, K), dtype=np.float16)
        A[np.arange(128), k0 + np.arange(128)] = 1.0
        want = (Q8[k0:k0 + 128].astype(np.float64) - 128) * np.ldexp(1.0, expo[k0 // G])[None, :]
        assert np.array_equal(layer(A).astype(np.float64), want)


def test_errors(marlin):
    import torch
    q = torch.zeros((256, 320), dtype=torch.uint8, device="cuda")
    s = torch.zeros((2, 320), dtype=torch.float16, device="cuda")
    with pytest.raises(marlin.MarlinError) as e:
        marlin.pack_w8(q, s, 128)
    assert e.value.status == 2
