"""GPU parity of the 2:4 sparse variant (marlin_pack_sparse24 / marlin_gemm_sparse24) through the C ABI."""
import numpy as np
import pytest

from paper_2408_11743_b200 import inputs
from gpu_util import DenseLayer, SparseLayer, to_dev, to_host

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def marlin():
    import torch
    assert torch.cuda.is_available()
    import paper_2408_11743_b200 as m
    m.lib()
    return m


def _codes(qk):
    out = np.zeros((qk.shape[0] * 8, qk.shape[1]), dtype=np.uint8)
    for j in range(8):
        out[j::8] = (qk >> np.uint32(4 * j)) & 15
    return out


@pytest.mark.parametrize("K,N,G", [(128, 64, 128), (256, 192, 128), (512, 320, 256), (2048, 1024, -1), (8192, 512, 128)])
def test_sparse_pack_matches_layout_reference_and_round_trips(marlin, K, N, G):
    from oracle import layout_ref
    case = inputs.make_sparse24(1, K, N, G, seed=K + N)
    w, meta, s = marlin.pack_sparse24(to_dev(case.qc_kpacked), to_dev(case.idx), to_dev(case.S), G)
    assert w.numel() == K * N // 4 and meta.numel() == K * N // 8
    assert np.array_equal(to_host(w).view(np.uint32), layout_ref.pack_sparse_codes(_codes(case.qc_kpacked), K))
    assert np.array_equal(to_host(meta).view(np.uint32), layout_ref.pack_sparse_meta(case.idx, K))
    assert np.array_equal(to_host(s).view(np.uint16), layout_ref.pack_scales(case.S).view(np.uint16).reshape(-1))
    qc2, idx2, s2 = marlin.unpack_sparse24(w, meta, s, K, N, G)
    assert np.array_equal(to_host(qc2).view(np.uint32), case.qc_kpacked)
    assert np.array_equal(to_host(idx2), case.idx)
    assert np.array_equal(to_host(s2).view(np.uint16), case.S.view(np.uint16))


SHAPES = [(1, 128, 64, 128), (3, 256, 192, 128), (8, 512, 128, -1), (16, 1024, 256, 128), (13, 2048, 512, -1),
          (16, 4096, 4096, 128), (17, 1024, 768, 128), (32, 2048, 1024, 128), (31, 1152, 448, 128),
          (33, 1024, 512, 128), (64, 2048, 1024, 128), (100, 1024, 640, -1), (128, 2048, 2048, 128),
          (5, 11008, 256, 128), (16, 8192, 8192, 128)]


@pytest.mark.parametrize("M,K,N,G", SHAPES)
def test_sparse_gemm_matches_oracle(marlin, oracle_lib, M, K, N, G):
    case = inputs.make_sparse24(M, K, N, G, seed=2000 + M + K + N)
    C = SparseLayer(marlin, case, M)(case.A)
    C_ref = oracle_lib.gemm_sparse24(case.A, case.qc_kpacked, case.idx, case.S, case.G)
    bad, worst, rms = oracle_lib.check_tolerance(C, C_ref)
    assert bad == 0, f"{bad} elements out of tolerance, worst ratio {worst:.3f}, rms {rms:.3f}"


# the partition and the fix-up the planner did not pick for a shape, forced through the library's tuning switches
SPARSE_MODES = [{"MARLIN_B200_SPLIT": "0", "MARLIN_B200_TC_SPLIT": "0"}, {"MARLIN_B200_CLUSTER": "0", "MARLIN_B200_TC_CLUSTER": "0"},
                {"MARLIN_B200_NW": "1"}, {"MARLIN_B200_NW": "2"}, {"MARLIN_B200_NW": "4", "MARLIN_B200_SPLIT": "0"},
                {"MARLIN_B200_CW": "12"}, {"MARLIN_B200_CW": "12", "MARLIN_B200_NW": "1", "MARLIN_B200_SPLIT": "0"},
                {"MARLIN_B200_CW": "12", "MARLIN_B200_NW": "2", "MARLIN_B200_CLUSTER": "0"}]


@pytest.mark.parametrize("mode", range(len(SPARSE_MODES)))
def test_sparse_every_partition_and_fixup_path(marlin, oracle_lib, mode, monkeypatch):
    for k, v in SPARSE_MODES[mode].items():
        monkeypatch.setenv(k, v)
    for M, K, N, G in [(1, 4096, 4096, 128), (8, 2048, 1536, 128), (16, 1024, 768, -1), (40, 4096, 1024, 128),
                       (8, 2048, 1344, 128), (16, 1024, 704, -1), (40, 4096, 320, 128), (128, 2048, 2048, 128),
                       (64, 8192, 1024, -1)]:
        case = inputs.make_sparse24(M, K, N, G, seed=17 * mode + M + K + N)
        C = SparseLayer(marlin, case, M)(case.A)
        C_ref = oracle_lib.gemm_sparse24(case.A, case.qc_kpacked, case.idx, case.S, case.G)
        bad, worst, rms = oracle_lib.check_tolerance(C, C_ref)
        assert bad == 0, f"{bad} elements out of tolerance, worst ratio {worst:.3f}, rms {rms:.3f}"


@pytest.mark.parametrize("M,K,N,exact", [
    (1, 4096, 4096, False),     # wide layout (N a multiple of 256): tcgen05.mma.sp kernel, partial tiles added at the L2
    (16, 4096, 22016, False),
    (64, 8192, 8192, True),     # tcgen05.mma.sp kernel, clusters: fixed order of the sum
    (40, 2048, 1024, False),
    (8, 4096, 1344, True),      # N = 64 mod 256: warp-level mma.sp kernel, fixed order of the sum
    (40, 2048, 448, True),      # the same in slabs of 16 rows
])
def test_sparse_long_stream_of_overlapping_launches_is_stable(marlin, oracle_lib, M, K, N, exact):
    # 120 launches that overlap on the stream and share one workspace, two inputs and two outputs in turn:
    # at the end each output holds what a single launch gives (bit for bit where the order of the sum is fixed;
    # within a quarter of the allowance where partial tiles are added at the L2 in arrival order)
    import torch
    case = inputs.make_sparse24(M, K, N, 128, seed=9 + M)
    other = inputs.make_sparse24(M, K, N, 128, seed=10 + M)
    layer = SparseLayer(marlin, case, M)
    A = [to_dev(case.A), to_dev(other.A)]
    want = [layer(case.A).copy(), layer(other.A).copy()]
    C = [torch.empty((M, N), dtype=torch.float16, device="cuda") for _ in range(2)]
    for rep in range(2):
        for c in C:
            c.fill_(float("nan"))
        for i in range(120):
            marlin.gemm_sparse24(A[i % 2], layer.w, layer.meta, layer.s, K, N, 128, layer.ws, out=C[i % 2])
        torch.cuda.synchronize()
        assert marlin.read_status(layer.ws) == 0
        for i in range(2):
            got = to_host(C[i])
            if exact:
                assert np.array_equal(got.view(np.uint16), want[i].view(np.uint16)), f"repetition {rep}, buffer {i}"
            else:
                bad, worst, _ = oracle_lib.check_tolerance(got, want[i])
                assert bad == 0 and worst < 0.25, f"repetition {rep}, buffer {i}"
    ws = to_host(layer.ws)
    assert np.all(ws[256:8192] == 0)   # arrival counters left clean


def test_sparse_equals_dense_kernel_on_the_expanded_matrix(marlin, oracle_lib):
    # the dense kernel on the matrix with code 8 (value 0) at the pruned positions computes the same layer
    M, K, N, G = 16, 2048, 1024, 128
    case = inputs.make_sparse24(M, K, N, G, seed=31)
    Q = oracle_lib.sparse24_expand(case.qc_kpacked, case.idx)
    dense = DenseLayer(marlin, inputs.kpack(Q), case.S, G, max_M=M)(case.A)
    sparse = SparseLayer(marlin, case, M)(case.A)
    C_ref = oracle_lib.gemm_sparse24(case.A, case.qc_kpacked, case.idx, case.S, G)
    assert oracle_lib.check_tolerance(sparse, C_ref)[0] == 0
    assert oracle_lib.check_tolerance(dense, C_ref)[0] == 0
    bad, worst, _ = oracle_lib.check_tolerance(sparse, dense)
    assert bad == 0 and worst < 0.3


@pytest.mark.parametrize("M,N", [(8, 256), (8, 192), (40, 512), (128, 256), (64, 320)])
def test_sparse_integer_closed_form_and_one_hot(marlin, oracle_lib, M, N):
    # N = 256, 512: the wide layout and the tcgen05.mma.sp kernel (its metadata placement in tensor memory is what the
    # one-hot rows probe); N = 192, 320: the warp-level mma.sp kernel
    rng = np.random.default_rng(8)
    K, G = 1024, 128
    case = inputs.make_sparse24(M, K, N, G, seed=9)
    case.A = rng.integers(-3, 4, size=(M, K)).astype(np.float16)
    case.S = np.ldexp(1.0, rng.integers(-4, 1, size=(K // G, N))).astype(np.float16)
    C = SparseLayer(marlin, case, M)(case.A)
    C_ref = oracle_lib.gemm_sparse24(case.A, case.qc_kpacked, case.idx, case.S, G)
    assert np.array_equal(C.view(np.uint16), C_ref.view(np.uint16))  # integers: exact in any order
    # one-hot rows read back single weights (0 at pruned positions), for every k of a few k-blocks
    Q = oracle_lib.sparse24_expand(case.qc_kpacked, case.idx)
    layer = SparseLayer(marlin, case, 128)
    for k0 in (0, 384, 896):
        A = np.zeros((128, K), dtype=np.float16)
        A[np.arange(128), k0 + np.arange(128)] = 1.0
        got = layer(A).astype(np.float64)
        want = (Q[k0:k0 + 128].astype(np.float64) - 8) * case.S[k0 // G].astype(np.float64)[None, :]
        assert np.array_equal(got, want)


def test_config5_full_size_on_sampled_outputs(marlin, oracle_lib):
    name, M, K, N, G, seed = list(inputs.iter_cases(5))[0]
    case = inputs.make_sparse24(M, K, N, G, seed)
    C = SparseLayer(marlin, case, M)(case.A)
    rng = np.random.default_rng(3)
    ms, ns = rng.integers(0, M, 2048), rng.integers(0, N, 2048)
    Q = oracle_lib.sparse24_expand(case.qc_kpacked, case.idx)
    ref = oracle_lib.gemm_samples(case.A, inputs.kpack(Q), case.S, G, ms, ns)
    bad, worst, _ = oracle_lib.check_tolerance(np.ascontiguousarray(C[ms, ns]), ref)
    assert bad == 0, worst
