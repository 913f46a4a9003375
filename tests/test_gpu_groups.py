"""GPU parity for scale groups of 64 and 32 rows (Section 2.3: group quantization; the paper's kernel section uses
one scale per 128 rows or per column, its discussion names smaller groups as an extension).

Such layers need N to be a multiple of 256 and run on the tcgen05 kernel at every batch size (dense and 2:4): the
two or four scale rows of a k-block travel with its weights, and every converted weight is multiplied by the scale
of its own 32-row quarter.  Bound: |C - C_ref| <= 5e-3 * (|C_ref| + rms(C_ref)); closed forms bit for bit.
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


SHAPES = [(1, 256, 256), (7, 1024, 512), (16, 4096, 4096), (33, 1024, 768), (64, 2048, 1024), (128, 4096, 2048),
          (200, 512, 256), (16, 11008, 256)]


@pytest.mark.parametrize("G", [64, 32])
@pytest.mark.parametrize("M,K,N", SHAPES)
def test_dense_small_groups_match_oracle(marlin, oracle_lib, M, K, N, G):
    case = inputs.make_dense(M, K, N, G, seed=7000 + M + K + N + G)
    C = DenseLayer(marlin, case.q_kpacked, case.S, G, max_M=M)(case.A)
    bad, worst, rms = oracle_lib.check_tolerance(C, oracle_lib.gemm(case.A, case.q_kpacked, case.S, G))
    assert bad == 0, f"{bad} elements out of tolerance, worst ratio {worst:.3f}, rms {rms:.3f}"


@pytest.mark.parametrize("G", [64, 32])
@pytest.mark.parametrize("M,K,N", [(8, 1024, 256), (40, 2048, 512), (128, 1024, 1024)])
def test_sparse_small_groups_match_oracle(marlin, oracle_lib, M, K, N, G):
    import torch
    case = inputs.make_sparse24(M, K, N, G, seed=7100 + M + K + N + G)
    w, meta, s = marlin.pack_sparse24(to_dev(case.qc_kpacked), to_dev(case.idx), to_dev(case.S), G)
    qc2, idx2, s2 = marlin.unpack_sparse24(w, meta, s, K, N, G)
    assert np.array_equal(to_host(qc2).view(np.uint32), case.qc_kpacked) and np.array_equal(to_host(idx2), case.idx)
    assert np.array_equal(to_host(s2).view(np.uint16), case.S.view(np.uint16))
    ws = marlin.new_workspace(M, K, N)
    C = to_host(marlin.gemm_sparse24(to_dev(case.A), w, meta, s, K, N, G, ws))
    torch.cuda.synchronize()
    assert marlin.read_status(ws) == 0
    bad, worst, rms = oracle_lib.check_tolerance(C, oracle_lib.gemm_sparse24(case.A, case.qc_kpacked, case.idx, case.S, G))
    assert bad == 0, f"{bad} elements out of tolerance, worst ratio {worst:.3f}, rms {rms:.3f}"


@pytest.mark.parametrize("G", [64, 32])
def test_small_groups_closed_form_and_one_hot(marlin, oracle_lib, G):
    # every (group, column) gets a power of two of its own: a row of scales used for the wrong quarter of a
    # k-block, or for the wrong column, shows as a wrong entry; integer activations make the sums exact
    K, N = 512, 256
    rng = np.random.default_rng(G)
    Q = rng.integers(0, 16, size=(K, N), dtype=np.uint8)
    expo = rng.integers(-6, 3, size=(K // G, N))
    S = np.ldexp(1.0, expo).astype(np.float16)
    q = inputs.kpack(Q)
    layer = DenseLayer(marlin, q, S, G, max_M=128)
    for k0 in range(0, K, 128):
        A = np.zeros((128, K), dtype=np.float16)
        A[np.arange(128), k0 + np.arange(128)] = 1.0
        want = (Q[k0:k0 + 128].astype(np.float64) - 8) * np.ldexp(1.0, expo[(k0 + np.arange(128)) // G])
        assert np.array_equal(layer(A).astype(np.float64), want), f"k-block {k0 // 128}"
    A = rng.integers(-3, 4, size=(24, K)).astype(np.float16)
    assert np.array_equal(layer(A).view(np.uint16), oracle_lib.gemm(A, q, S, G).view(np.uint16))


def test_small_groups_need_n_multiple_of_256(marlin):
    case = inputs.make_dense(4, 256, 192, 64, seed=1)
    with pytest.raises(marlin.MarlinError) as e:
        marlin.pack(to_dev(case.q_kpacked), to_dev(case.S), 64)
    assert e.value.status == 3
