"""marlin_quantize_rtn on the GPU against the CPU oracle (oracle/quantize_oracle.c): codes, scales bit for bit
(integers decided by fp32 arithmetic in a fixed order on both sides), then the whole chain quantise -> pack -> layer."""
import numpy as np
import pytest

from gpu_util import to_dev, to_host

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def marlin():
    import torch
    assert torch.cuda.is_available()
    import paper_2408_11743_b200 as m
    m.lib()
    return m


def _weights(K, N, seed, outliers=True):
    rng = np.random.default_rng(seed)
    W = (rng.standard_normal((K, N)) * rng.uniform(0.005, 0.05, size=(1, N))).astype(np.float16)
    if outliers:
        W[rng.integers(0, K, K // 16), rng.integers(0, N, K // 16)] *= 7
    W[:, 3] = 0                      # a column of zero groups
    W[5, 7] = np.float16(6.0e-8)     # a subnormal
    return W


@pytest.mark.parametrize("K,N,G,n_grid,n_cand", [
    (256, 64, 128, 20, 10), (1024, 320, 128, 20, 10), (512, 256, 64, 20, 10), (512, 512, 32, 16, 16),
    (768, 192, 256, 20, 1), (2048, 128, -1, 10, 5), (1152, 448, 384, 7, 3), (4096, 4096, 128, 20, 10)])
def test_codes_and_scales_match_the_oracle_bit_for_bit(marlin, K, N, G, n_grid, n_cand):
    import torch
    from oracle import quantize_ref
    from paper_2408_11743_b200 import inputs
    W = _weights(K, N, K + N + n_cand)
    Gn = K if G == -1 else G
    q, s = marlin.quantize_rtn(to_dev(W), G, n_grid, n_cand)
    torch.cuda.synchronize()
    Q_ref, S_ref, _ = quantize_ref.quantize_rtn(W, Gn, n_grid, n_cand)
    assert np.array_equal(to_host(s).view(np.uint16), S_ref.view(np.uint16))
    assert np.array_equal(to_host(q).view(np.uint32), inputs.kpack(Q_ref))


def test_plain_rounding_versus_search_on_outlier_groups(marlin):
    import torch
    W = _weights(1024, 256, 9, outliers=False)
    W[::128, :] *= 3
    Wd = W.astype(np.float64)

    def sq_err(n_cand):
        from oracle import unpack_q
        q, s = marlin.quantize_rtn(to_dev(W), 128, 20, n_cand)
        torch.cuda.synchronize()
        Q = unpack_q(to_host(q).view(np.uint32)).astype(np.float64)
        return ((Wd - (Q - 8) * np.repeat(to_host(s).astype(np.float64), 128, axis=0)) ** 2).sum()
    assert sq_err(10) < 0.9 * sq_err(1)


@pytest.mark.parametrize("M", [4, 48, 300])
def test_quantise_pack_layer_chain_is_close_to_the_fp16_product(marlin, oracle_lib, M):
    # the whole front end: fp16 weights -> codes and scales -> packed layer -> product, against (a) the oracle run on the
    # same codes and scales (the parity bound) and (b) the fp64 product with the unquantised weights (4-bit error level)
    import torch
    K, N, G = 2048, 512, 128
    W = _weights(K, N, 77, outliers=False)
    rng = np.random.default_rng(1)
    A = rng.standard_normal((M, K)).astype(np.float16)
    q, s = marlin.quantize_rtn(to_dev(W), G)
    w_packed, s_packed = marlin.pack(q, s, G)
    ws = marlin.new_workspace(M, K, N)
    C = to_host(marlin.gemm(to_dev(A), w_packed, s_packed, K, N, G, ws))
    torch.cuda.synchronize()
    assert marlin.read_status(ws) == 0
    C_ref = oracle_lib.gemm(A, to_host(q).view(np.uint32), to_host(s), G)
    bad, worst, _ = oracle_lib.check_tolerance(C, C_ref)
    assert bad == 0, worst
    exact = A.astype(np.float64) @ W.astype(np.float64)
    rel = np.linalg.norm(C.astype(np.float64) - exact) / np.linalg.norm(exact)
    assert rel < 0.12, rel  # uniform 4-bit grid over Gaussian groups of 128: about 8-9 % relative error


def test_argument_checks(marlin):
    import torch
    W = torch.zeros((256, 64), dtype=torch.float16, device="cuda")
    with pytest.raises(marlin.MarlinError):
        marlin.quantize_rtn(W, 100)
    with pytest.raises(marlin.MarlinError) as e:
        marlin.quantize_rtn(W, 128, 4, 5)
    assert e.value.status == 2
    with pytest.raises(marlin.MarlinError):
        marlin.quantize_rtn(torch.zeros((250, 64), dtype=torch.float16, device="cuda"), 128)
