"""GPU parity of marlin_gemm against the CPU oracle, through the C ABI.

Bound (floating point): |C - C_ref| <= 5e-3 * (|C_ref| + rms(C_ref)) for every element.
Integer-valued closed forms must match bit for bit.
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


def _assert_close(oracle_lib, C, C_ref):
    bad, worst, rms = oracle_lib.check_tolerance(C, C_ref)
    assert bad == 0, f"{bad} elements out of tolerance, worst ratio {worst:.3f}, rms {rms:.3f}"
    return worst


# small shapes the oracle finishes at once; several tiles, ragged M, both scale modes,
# K and N that are not multiples of the wide tiles, shapes with fewer units than SMs
SMALL = [
    (1, 128, 64, 128), (2, 256, 64, 128), (5, 256, 192, 128), (8, 512, 128, -1), (3, 384, 320, 128),
    (16, 1024, 256, 128), (9, 1024, 384, 256), (13, 2048, 512, -1), (16, 4096, 4096, 128),
    (17, 1024, 768, 128), (32, 2048, 1024, 128), (31, 1152, 448, 128), (24, 4096, 1024, -1),
    (33, 1024, 512, 128), (64, 2048, 1024, 128), (100, 1024, 640, -1), (128, 2048, 2048, 128),
    (7, 11008, 256, 128), (1, 8192, 8192, 128), (4, 4096, 12288, 128), (16, 28672, 1024, -1),
    (16, 28672, 1024, 128), (32, 4096, 22016, 128),
    # groups of three k-blocks (no power of two), in both kernels; more rows than one launch takes
    (8, 1152, 256, 384), (40, 1152, 512, 384), (200, 1024, 512, 128), (150, 512, 192, 128),
]


@pytest.mark.parametrize("M,K,N,G", SMALL)
def test_gemm_matches_oracle(marlin, oracle_lib, M, K, N, G):
    case = inputs.make_dense(M, K, N, G, seed=1000 + M + K + N)
    layer = DenseLayer(marlin, case.q_kpacked, case.S, G, max_M=M)
    C = layer(case.A)
    C_ref = oracle_lib.gemm(case.A, case.q_kpacked, case.S, case.G)
    _assert_close(oracle_lib, C, C_ref)


# The planner picks a partition and a fix-up per shape, so the default run exercises only one of them for a
# given shape.  The tuning switches of the library force the others: even stripes instead of the tile-aligned
# partition, the workspace fix-up instead of thread-block clusters, each tile width.
MODES = [
    {"MARLIN_B200_SPLIT": "0", "MARLIN_B200_TC_SPLIT": "0"},             # even stripes in both kernels
    {"MARLIN_B200_CLUSTER": "0", "MARLIN_B200_TC_CLUSTER": "0"},         # no clusters: fix-up through the workspace
    {"MARLIN_B200_NW": "1"}, {"MARLIN_B200_NW": "2"}, {"MARLIN_B200_NW": "4"},
    {"MARLIN_B200_NW": "4", "MARLIN_B200_SPLIT": "0"}, {"MARLIN_B200_NW": "1", "MARLIN_B200_CLUSTER": "0"},
    # twelve consumer warps (the planner takes them on long stripes only) in every tile width, partition and fix-up
    {"MARLIN_B200_CW": "12"}, {"MARLIN_B200_CW": "12", "MARLIN_B200_NW": "1", "MARLIN_B200_CLUSTER": "0"},
    {"MARLIN_B200_CW": "12", "MARLIN_B200_NW": "2", "MARLIN_B200_SPLIT": "0"}, {"MARLIN_B200_CW": "12", "MARLIN_B200_NW": "4"},
    {"MARLIN_B200_CW": "8"},
    # the cluster exchange through the first CTA's stage ring (two cluster barriers) instead of a buffer behind the ring
    {"MARLIN_B200_XBUF": "0"}, {"MARLIN_B200_XBUF": "0", "MARLIN_B200_CW": "12", "MARLIN_B200_NW": "2"},
]
MODE_SHAPES = [(1, 4096, 4096, 128), (8, 2048, 1536, 128), (16, 1024, 768, -1), (13, 11008, 512, 128),
               (40, 4096, 4096, 128), (128, 2048, 1024, 128), (64, 8192, 8192, 128)]


@pytest.mark.parametrize("mode", range(len(MODES)))
def test_every_partition_and_fixup_path_matches_oracle(marlin, oracle_lib, mode, monkeypatch):
    for k, v in MODES[mode].items():
        monkeypatch.setenv(k, v)
    for M, K, N, G in MODE_SHAPES:
        case = inputs.make_dense(M, K, N, G, seed=31 * mode + M + K + N)
        layer = DenseLayer(marlin, case.q_kpacked, case.S, G, max_M=M)
        C = layer(case.A)
        _assert_close(oracle_lib, C, oracle_lib.gemm(case.A, case.q_kpacked, case.S, case.G))
        counters = to_host(layer.ws[256:8192])
        assert np.all(counters == 0)


def test_config1_single_layer(marlin, oracle_lib):
    name, M, K, N, G, seed = next(inputs.iter_cases(1))
    case = inputs.make_dense(M, K, N, G, seed)
    C = DenseLayer(marlin, case.q_kpacked, case.S, G, max_M=M)(case.A)
    worst = _assert_close(oracle_lib, C, oracle_lib.gemm(case.A, case.q_kpacked, case.S, G))
    assert worst < 0.5  # an honest fp32-accumulating kernel sits far inside the bound


def test_same_layer_many_batch_sizes_and_repeatability(marlin, oracle_lib):
    K, N, G = 2048, 1536, 128
    case = inputs.make_dense(128, K, N, G, seed=77)
    layer = DenseLayer(marlin, case.q_kpacked, case.S, G, max_M=128)
    C_ref = oracle_lib.gemm(case.A, case.q_kpacked, case.S, G)
    for M in (1, 2, 3, 4, 7, 8, 9, 15, 16, 17, 31, 32, 33, 63, 64, 65, 127, 128):
        C = layer(case.A[:M])
        # rows are independent: the reference of the first M rows is the first M rows of the reference,
        # but the bound's rms is over the compared block
        _assert_close(oracle_lib, C, np.ascontiguousarray(C_ref[:M]))
        C2 = layer(case.A[:M])
        if M <= 16:
            # warp-MMA kernel: partial tiles are summed in stripe order, the result is reproducible bit for bit
            assert np.array_equal(C.view(np.uint16), C2.view(np.uint16))
        else:
            # tcgen05 kernel: shared tiles are summed by L2 reductions in arrival order (fp32): equal up to
            # the last bit of the fp16 result (one fp16 ulp is up to ~0.1 of the allowance here)
            bad, worst, _ = oracle_lib.check_tolerance(C2, C)
            assert bad == 0 and worst < 0.25


@pytest.mark.parametrize("M,K,N,exact", [
    (1, 4096, 4096, True),      # tile-aligned, two k-ranges per tile: thread-block clusters
    (16, 2048, 8192, True),     # one CTA per tile, no fix-up
    (8, 4096, 22016, True),     # even stripes, workspace fix-up, mid-stripe segments
    (64, 8192, 8192, True),     # tcgen05 kernel, clusters of four
    (40, 4096, 4096, False),    # tcgen05 kernel, L2 reductions (arrival order: last bit may differ)
])
def test_a_long_stream_of_overlapping_launches_is_stable(marlin, oracle_lib, M, K, N, exact):
    # Consecutive launches overlap (the next kernel starts its prologue and its weight copies while the previous
    # one drains) and share one workspace.  120 launches alternating two inputs and two outputs must give, at
    # the end, exactly what a single launch gives.
    import torch
    case0 = inputs.make_dense(M, K, N, 128, seed=5 + M)
    case1 = inputs.make_dense(M, K, N, 128, seed=6 + M)
    layer = DenseLayer(marlin, case0.q_kpacked, case0.S, 128, max_M=M)
    A = [to_dev(case0.A), to_dev(case1.A)]
    want = []
    for a in A:
        want.append(to_host(marlin.gemm(a, layer.w, layer.s, K, N, 128, layer.ws)).copy())
        torch.cuda.synchronize()
    C = [torch.empty((M, N), dtype=torch.float16, device="cuda") for _ in range(2)]
    for rep in range(3):
        for c in C:
            c.fill_(float("nan"))
        for i in range(120):
            marlin.gemm(A[i % 2], layer.w, layer.s, K, N, 128, layer.ws, out=C[i % 2])
        torch.cuda.synchronize()
        assert marlin.read_status(layer.ws) == 0
        for i in range(2):
            got = to_host(C[i])
            if exact:
                assert np.array_equal(got.view(np.uint16), want[i].view(np.uint16)), f"repetition {rep}, buffer {i}"
            else:
                bad, worst, _ = oracle_lib.check_tolerance(got, want[i])
                assert bad == 0 and worst < 0.25
    _assert_close(oracle_lib, to_host(C[0]), oracle_lib.gemm(case0.A, case0.q_kpacked, case0.S, 128))


def test_zero_codes_give_zero(marlin):
    K, N = 1024, 256
    q = inputs.kpack(np.full((K, N), 8, dtype=np.uint8))
    case = inputs.make_dense(5, K, N, 128, seed=3)
    C = DenseLayer(marlin, q, case.S, 128, max_M=5)(case.A)
    assert np.all(C == 0)


@pytest.mark.parametrize("M,K,N", [(2, 4096, 256), (16, 8192, 512), (32, 2048, 320)])
def test_integer_closed_form_is_bit_exact(marlin, oracle_lib, M, K, N):
    # scales are powers of two and activations small integers: every product and every partial sum is
    # an integer multiple of the scale below 2^24, so fp32 accumulation in any order is exact and the
    # GPU must equal the oracle bit for bit
    rng = np.random.default_rng(M + K)
    Q = rng.integers(0, 16, size=(K, N), dtype=np.uint8)
    A = rng.integers(-3, 4, size=(M, K)).astype(np.float16)
    S = np.ldexp(1.0, rng.integers(-4, 1, size=(K // 128, N))).astype(np.float16)
    q = inputs.kpack(Q)
    C = DenseLayer(marlin, q, S, 128, max_M=M)(A)
    C_ref = oracle_lib.gemm(A, q, S, 128)
    assert np.array_equal(C.view(np.uint16), C_ref.view(np.uint16))
    # all-ones row and unit scales: plain column sums of (Q - 8)
    A1 = np.ones((1, K), dtype=np.float16)
    S1 = np.ones((1, N), dtype=np.float16)
    C1 = DenseLayer(marlin, q, S1, K, max_M=1)(A1)
    assert np.array_equal(C1.view(np.uint16), oracle_lib.gemm(A1, q, S1, K).view(np.uint16))


def test_one_hot_rows_probe_every_k_position(marlin, oracle_lib):
    # A = unit vectors e_k: C[m, n] = (Q[k_m, n] - 8) * S[k_m // G, n] exactly; sweeps every k
    K, N, G = 512, 192, 128
    rng = np.random.default_rng(5)
    Q = rng.integers(0, 16, size=(K, N), dtype=np.uint8)
    expo = rng.integers(-5, 2, size=(K // G, N))
    S = np.ldexp(1.0, expo).astype(np.float16)
    q = inputs.kpack(Q)
    layer = DenseLayer(marlin, q, S, G, max_M=128)
    for k0 in range(0, K, 128):
        A = np.zeros((128, K), dtype=np.float16)
        A[np.arange(128), k0 + np.arange(128)] = 1.0
        C = layer(A).astype(np.float64)
        want = (Q[k0:k0 + 128].astype(np.float64) - 8) * np.ldexp(1.0, expo[(k0 // G)])[None, :]
        assert np.array_equal(C, want)


# Exact-answer tests on the large-batch kernels (17 rows and more per launch), in every partition and fix-up
# those kernels have: the default, even stripes, and the reduction through the workspace instead of clusters.
LARGE_BATCH_MODES = [{}, {"MARLIN_B200_TC_SPLIT": "0", "MARLIN_B200_SPLIT": "0"},
                     {"MARLIN_B200_TC_CLUSTER": "0", "MARLIN_B200_CLUSTER": "0"}]


@pytest.mark.parametrize("mode", range(len(LARGE_BATCH_MODES)))
@pytest.mark.parametrize("M,K,N,G", [(33, 1024, 256, 128), (64, 2048, 512, 128), (128, 4096, 1024, -1),
                                     (17, 1024, 512, 256), (48, 2048, 256, -1)])
def test_integer_closed_form_is_bit_exact_on_the_large_batch_kernels(marlin, oracle_lib, monkeypatch, mode, M, K, N, G):
    # powers of two as scales and small integers as activations: every product and every partial sum is an
    # integer multiple of the scale below 2^24, so fp32 sums are exact in ANY order (also the arrival order of
    # the reductions at the L2) and the result must equal the oracle bit for bit
    for k, v in LARGE_BATCH_MODES[mode].items():
        monkeypatch.setenv(k, v)
    rng = np.random.default_rng(7 * M + K + N)
    Q = rng.integers(0, 16, size=(K, N), dtype=np.uint8)
    A = rng.integers(-3, 4, size=(M, K)).astype(np.float16)
    Gn = K if G == -1 else G
    S = np.ldexp(1.0, rng.integers(-4, 1, size=(K // Gn, N))).astype(np.float16)
    q = inputs.kpack(Q)
    C = DenseLayer(marlin, q, S, G, max_M=M)(A)
    C_ref = oracle_lib.gemm(A, q, S, Gn)
    assert np.array_equal(C.view(np.uint16), C_ref.view(np.uint16))


@pytest.mark.parametrize("mode", range(len(LARGE_BATCH_MODES)))
@pytest.mark.parametrize("N", [256, 512])
def test_one_hot_rows_probe_every_k_position_on_the_large_batch_kernels(marlin, monkeypatch, mode, N):
    # 128 unit vectors at a time: C[m, n] = (Q[k_m, n] - 8) * S[k_m // G, n] exactly, for every k of the layer;
    # a wrong operand descriptor, k order or scale group shows as a wrong entry
    for k, v in LARGE_BATCH_MODES[mode].items():
        monkeypatch.setenv(k, v)
    K, G = 1024, 128
    rng = np.random.default_rng(11 + N)
    Q = rng.integers(0, 16, size=(K, N), dtype=np.uint8)
    expo = rng.integers(-5, 2, size=(K // G, N))
    S = np.ldexp(1.0, expo).astype(np.float16)
    layer = DenseLayer(marlin, inputs.kpack(Q), S, G, max_M=128)
    for k0 in range(0, K, 128):
        A = np.zeros((128, K), dtype=np.float16)
        A[np.arange(128), k0 + np.arange(128)] = 1.0
        C = layer(A).astype(np.float64)
        want = (Q[k0:k0 + 128].astype(np.float64) - 8) * np.ldexp(1.0, expo[k0 // G])[None, :]
        assert np.array_equal(C, want), f"k-block {k0 // 128}"
    # the same with fewer rows (other instances of the kernels): rows = the first 40 / 64 unit vectors of a block
    for M in (40, 64):
        A = np.zeros((M, K), dtype=np.float16)
        A[np.arange(M), 300 + np.arange(M)] = 1.0
        want = np.stack([(Q[300 + i].astype(np.float64) - 8) * np.ldexp(1.0, expo[(300 + i) // G]) for i in range(M)])
        assert np.array_equal(layer(A).astype(np.float64), want), f"M = {M}"


def test_subnormal_scales_and_large_values(marlin, oracle_lib):
    K, N = 1024, 128
    case = inputs.make_dense(4, K, N, 128, seed=9)
    S = np.full((K // 128, N), 2.0 ** -20, dtype=np.float16)  # subnormal fp16
    C = DenseLayer(marlin, case.q_kpacked, S, 128, max_M=4)(case.A)
    _assert_close(oracle_lib, C, oracle_lib.gemm(case.A, case.q_kpacked, S, 128))
    S = np.full((K // 128, N), 4.0, dtype=np.float16)
    A = (case.A.astype(np.float32) * 8).astype(np.float16)
    C = DenseLayer(marlin, case.q_kpacked, S, 128, max_M=4)(A)
    _assert_close(oracle_lib, C, oracle_lib.gemm(A, case.q_kpacked, S, 128))


@pytest.mark.parametrize("M,G", [(1, 128), (8, 128), (8, -1), (16, 128), (32, 128)])
def test_activations_with_offset_and_outliers(marlin, oracle_lib, M, G):
    # The small-batch kernels carry the offsets of the exponent trick (1024 + q, 64 + q) through the product and take
    # them off per scale group: activations with a non-zero mean and a few outliers of 1e2..1e3 among small values make
    # those offset sums large against the result.  The bound must still hold, also on the columns whose reference
    # is small (their allowance is 5e-3 * rms alone).
    K, N = 4096, 512
    rng = np.random.default_rng(100 + M)
    A = (0.5 + 0.25 * rng.standard_normal((M, K))).astype(np.float32)
    for m in range(M):
        ks = rng.choice(K, size=6, replace=False)
        A[m, ks] = rng.choice([-1.0, 1.0], size=6) * rng.uniform(1e2, 1e3, size=6)
    A = A.astype(np.float16)
    case = inputs.make_dense(M, K, N, G, seed=200 + M)
    C = DenseLayer(marlin, case.q_kpacked, case.S, G, max_M=M)(A)
    C_ref = oracle_lib.gemm(A, case.q_kpacked, case.S, case.G)
    bad, worst, rms = oracle_lib.check_tolerance(C, C_ref)
    assert bad == 0, f"{bad} elements out of tolerance, worst ratio {worst:.3f}, rms {rms:.3f}"
    small = np.abs(C_ref.astype(np.float64)) < 0.05 * rms
    assert small.any()
    err = np.abs(C.astype(np.float64) - C_ref.astype(np.float64))
    assert err[small].max() <= 5e-3 * (0.05 * rms + rms)


@pytest.mark.parametrize("M", [4, 32, 128])
def test_scales_near_and_below_the_smallest_normal_half(marlin, oracle_lib, M):
    # scales around 2^-14 (the smallest normal fp16) and below: the large-batch kernel multiplies (q - 8) * s in fp16
    # before the MMA, where such products are subnormal; the result must still be within the bound of the exact one
    K, N = 2048, 512
    case = inputs.make_dense(M, K, N, 128, seed=300 + M)
    rng = np.random.default_rng(M)
    S = (2.0 ** -14 * rng.uniform(0.25, 2.0, size=(K // 128, N))).astype(np.float16)
    A = (case.A.astype(np.float32) * 16).astype(np.float16)
    C = DenseLayer(marlin, case.q_kpacked, S, 128, max_M=M)(A)
    bad, worst, rms = oracle_lib.check_tolerance(C, oracle_lib.gemm(A, case.q_kpacked, S, 128))
    assert bad == 0, f"{bad} elements out of tolerance, worst ratio {worst:.3f}, rms {rms:.3g}"


def test_full_size_layers_on_sampled_outputs(marlin, oracle_lib):
    # the largest layers of the workload list, checked on outputs the oracle computes one by one
    rng = np.random.default_rng(2)
    for (K, N, G, M) in [(8192, 57344, 128, 16), (28672, 8192, -1, 64), (8192, 8192, 128, 128)]:
        case = inputs.make_dense(M, K, N, G, seed=K + N + M)
        C = DenseLayer(marlin, case.q_kpacked, case.S, G, max_M=M)(case.A)
        ms = rng.integers(0, M, 4096)
        ns = rng.integers(0, N, 4096)
        ref = oracle_lib.gemm_samples(case.A, case.q_kpacked, case.S, case.G, ms, ns)
        # the bound's rms is taken over the sampled outputs (a fair estimate of the full one)
        bad, worst, _ = oracle_lib.check_tolerance(np.ascontiguousarray(C[ms, ns]), ref)
        assert bad == 0, (K, N, G, M, worst)
        assert np.all(np.isfinite(C.astype(np.float32)))


def test_errors_and_status(marlin):
    import torch
    K, N = 256, 128
    case = inputs.make_dense(4, K, N, 128, seed=1)
    layer = DenseLayer(marlin, case.q_kpacked, case.S, 128, max_M=4)
    A = to_dev(case.A)
    small_ws = torch.zeros(1024, dtype=torch.uint8, device="cuda")
    with pytest.raises(marlin.MarlinError) as e:
        marlin.gemm(A, layer.w, layer.s, K, N, 128, small_ws)
    assert e.value.status == 5
    assert marlin.read_status(layer.ws) == 0
    # the arrival counters are left at zero by every call
    layer(case.A)
    counters = to_host(layer.ws[256:256 + 4096]).view(np.int32)
    assert np.all(counters == 0)


def test_workspace_is_clean_after_large_batch_calls(marlin, oracle_lib):
    # the tcgen05 kernel accumulates shared tiles in the workspace and must leave them zero for the next call
    K, N, G = 1024, 512, 128
    case = inputs.make_dense(128, K, N, G, seed=12)
    layer = DenseLayer(marlin, case.q_kpacked, case.S, G, max_M=128)
    C_ref = oracle_lib.gemm(case.A, case.q_kpacked, case.S, G)
    for M in (128, 40, 128, 64):
        C = layer(case.A[:M])
        _assert_close(oracle_lib, C, np.ascontiguousarray(C_ref[:M]))
        ws = to_host(layer.ws)
        assert np.all(ws[256:8192] == 0)                    # counters
        assert np.all(ws[-N * 128 * 4:] == 0)               # accumulation tiles (placed at the end)


def test_layer_object_makes_the_same_calls(marlin, oracle_lib):
    # Layer checks the packed buffers once and then makes the same foreign call as the functions: same results
    # (bit for bit where the kernel's summation order is fixed), same errors for a bad A
    import torch
    from oracle import w8_ref, zp_ref
    K, N, G, M = 1024, 512, 128, 8
    case = inputs.make_dense(M, K, N, G, seed=5)
    A = to_dev(case.A)
    w, s = marlin.pack(to_dev(case.q_kpacked), to_dev(case.S), G)
    ws = marlin.new_workspace(64, K, N)
    dense = marlin.Layer(w, s, K, N, G, ws, max_M=64)
    assert torch.equal(dense(A), marlin.gemm(A, w, s, K, N, G, ws))
    out = torch.empty((M, N), dtype=torch.float16, device="cuda")
    assert dense(A, out=out) is out
    call = dense.prepare(A, out=out)           # buffers checked once, the same foreign call on every use
    out.zero_()
    assert call() is out and torch.equal(out, marlin.gemm(A, w, s, K, N, G, ws))
    Z = np.random.default_rng(1).integers(0, 16, size=case.S.shape, dtype=np.uint8)
    z = marlin.pack_zeros(to_dev(Z), K, N, G)
    zp = marlin.Layer(w, s, K, N, G, ws, z_packed=z)
    assert torch.equal(zp(A), marlin.gemm_zp(A, w, s, z, K, N, G, ws))
    sp = inputs.make_sparse24(M, K, N, G, seed=6)
    w2, meta, s2 = marlin.pack_sparse24(to_dev(sp.qc_kpacked), to_dev(sp.idx), to_dev(sp.S), sp.G)
    sparse = marlin.Layer(w2, s2, K, N, G, ws, meta_packed=meta)
    bad, worst, _ = oracle_lib.check_tolerance(to_host(sparse(to_dev(sp.A))),
                                               oracle_lib.gemm_sparse24(sp.A, sp.qc_kpacked, sp.idx, sp.S, sp.G))
    assert bad == 0, worst
    rng = np.random.default_rng(7)
    Q8 = rng.integers(0, 256, size=(K, N), dtype=np.uint8)
    S8 = rng.uniform(0.0005, 0.002, size=(K // G, N)).astype(np.float16)
    w8, s8 = marlin.pack_w8(to_dev(Q8), to_dev(S8), G)
    eight = marlin.Layer(w8, s8, K, N, G, ws, w8=True)
    bad, worst, _ = oracle_lib.check_tolerance(to_host(eight(A)), w8_ref.gemm_w8(case.A, Q8, S8, G))
    assert bad == 0, worst
    torch.cuda.synchronize()
    assert marlin.read_status(ws) == 0
    with pytest.raises(ValueError):
        dense(A[:, :512])                       # wrong K (and not contiguous)
    with pytest.raises(ValueError):
        dense(A.float())
    with pytest.raises(ValueError):
        marlin.Layer(w, s, K, N, 64, ws)        # scale buffer does not match the group size
    with pytest.raises(ValueError):
        marlin.Layer(w, s, K, N, G, ws, max_M=100000)
