"""Seeded random walk over shapes, batch sizes, formats (dense, 2:4, zero points, 8-bit), group sizes and the
partition / fix-up switches: every case compared with its CPU oracle through the C ABI (the layer's bound
|C - C_ref| <= 5e-3 (|C_ref| + rms)), status word zero, arrival counters left at zero."""
import numpy as np
import pytest

from paper_2408_11743_b200 import inputs
from gpu_util import to_dev, to_host

pytestmark = pytest.mark.gpu

SWITCHES = ["MARLIN_B200_SPLIT", "MARLIN_B200_TC_SPLIT", "MARLIN_B200_CLUSTER", "MARLIN_B200_TC_CLUSTER", "MARLIN_B200_NW",
            "MARLIN_B200_CW"]
BATCHES = [1, 2, 3, 5, 8, 9, 13, 16, 17, 24, 32, 33, 48, 64, 65, 100, 128, 129, 200, 256, 300, 513]


@pytest.mark.parametrize("seed", [11, 12, 13])
def test_random_cases_match_their_oracles(oracle_lib, monkeypatch, seed):
    import torch
    import paper_2408_11743_b200 as marlin
    from oracle import w8_ref, zp_ref
    rng = np.random.default_rng(seed)
    done = 0
    while done < 120:
        for k in SWITCHES:
            monkeypatch.delenv(k, raising=False)
        mode = int(rng.integers(0, 6))
        if mode == 1:
            monkeypatch.setenv("MARLIN_B200_SPLIT", "0")
            monkeypatch.setenv("MARLIN_B200_TC_SPLIT", "0")
        elif mode == 2:
            monkeypatch.setenv("MARLIN_B200_CLUSTER", "0")
            monkeypatch.setenv("MARLIN_B200_TC_CLUSTER", "0")
        elif mode == 3:
            monkeypatch.setenv("MARLIN_B200_NW", str(rng.choice([1, 2, 4])))
        elif mode == 4:
            monkeypatch.setenv("MARLIN_B200_TC_SPLIT", str(rng.choice([2, 4, 8])))
        if rng.integers(0, 3) == 0:
            monkeypatch.setenv("MARLIN_B200_CW", "12")   # twelve consumer warps wherever the batch allows them
        fmt = str(rng.choice(["dense", "dense", "sparse", "zp", "w8"]))
        K = 128 * int(rng.integers(1, 40))
        nmul = 256 if fmt == "w8" else 64
        N = nmul * int(rng.integers(1, 2048 // nmul + 1))
        M = int(rng.choice(BATCHES))
        groups = [-1, 128] + ([256] if K % 256 == 0 else []) + ([64, 32] if N % 256 == 0 else [])
        G = int(rng.choice(groups))
        Gn = K if G == -1 else G
        case_seed = int(rng.integers(0, 1 << 30))
        what = (fmt, M, K, N, G, mode)
        if fmt == "sparse":
            case = inputs.make_sparse24(M, K, N, G, seed=case_seed)
            w, meta, s = marlin.pack_sparse24(to_dev(case.qc_kpacked), to_dev(case.idx), to_dev(case.S), case.G)
            ws = marlin.new_workspace(M, K, N)
            C = to_host(marlin.gemm_sparse24(to_dev(case.A), w, meta, s, K, N, case.G, ws))
            ref = oracle_lib.gemm_sparse24(case.A, case.qc_kpacked, case.idx, case.S, case.G)
        elif fmt == "w8":
            r2 = np.random.default_rng(case_seed)
            Q8 = r2.integers(0, 256, size=(K, N), dtype=np.uint8)
            S = r2.uniform(0.0005, 0.002, size=(K // Gn, N)).astype(np.float16)
            A = r2.standard_normal((M, K)).astype(np.float16)
            w, s = marlin.pack_w8(to_dev(Q8), to_dev(S), G)
            ws = marlin.new_workspace(M, K, N)
            C = to_host(marlin.gemm_w8(to_dev(A), w, s, K, N, G, ws))
            ref = w8_ref.gemm_w8(A, Q8, S, Gn)
        else:
            case = inputs.make_dense(M, K, N, G, seed=case_seed)
            w, s = marlin.pack(to_dev(case.q_kpacked), to_dev(case.S), G)
            ws = marlin.new_workspace(M, K, N)
            if fmt == "zp":
                Z = np.random.default_rng(case_seed + 1).integers(0, 16, size=case.S.shape, dtype=np.uint8)
                z = marlin.pack_zeros(to_dev(Z), K, N, G)
                C = to_host(marlin.gemm_zp(to_dev(case.A), w, s, z, K, N, G, ws))
                ref = zp_ref.gemm_zp(case.A, case.q_kpacked, case.S, Z, case.G)
            else:
                C = to_host(marlin.gemm(to_dev(case.A), w, s, K, N, G, ws))
                ref = oracle_lib.gemm(case.A, case.q_kpacked, case.S, case.G)
        torch.cuda.synchronize()
        assert marlin.read_status(ws) == 0, what
        bad, worst, _ = oracle_lib.check_tolerance(C, ref)
        assert bad == 0, (what, worst)
        assert bool((ws[256:8192] == 0).all()), what
        done += 1


def _random_layer(rng, marlin, oracle_lib, max_rows):
    """A random packed layer of a random format: (call(A_dev, M, ws) -> C_dev, ref(M) -> C_ref, (K, N), description)."""
    from oracle import w8_ref, zp_ref
    fmt = str(rng.choice(["dense", "dense", "sparse", "zp", "w8"]))
    K = 128 * int(rng.integers(1, 24))
    nmul = 256 if fmt == "w8" else 64
    N = nmul * int(rng.integers(1, 1536 // nmul + 1))
    groups = [-1, 128] + ([256] if K % 256 == 0 else []) + ([64, 32] if N % 256 == 0 else [])
    G = int(rng.choice(groups))
    Gn = K if G == -1 else G
    seed = int(rng.integers(0, 1 << 30))
    what = (fmt, K, N, G)
    if fmt == "sparse":
        case = inputs.make_sparse24(max_rows, K, N, G, seed=seed)
        w, meta, s = marlin.pack_sparse24(to_dev(case.qc_kpacked), to_dev(case.idx), to_dev(case.S), case.G)
        A = case.A
        call = lambda Ad, ws: marlin.gemm_sparse24(Ad, w, meta, s, K, N, case.G, ws)
        ref = lambda M: oracle_lib.gemm_sparse24(np.ascontiguousarray(A[:M]), case.qc_kpacked, case.idx, case.S, case.G)
    elif fmt == "w8":
        r2 = np.random.default_rng(seed)
        Q8 = r2.integers(0, 256, size=(K, N), dtype=np.uint8)
        S = r2.uniform(0.0005, 0.002, size=(K // Gn, N)).astype(np.float16)
        A = r2.standard_normal((max_rows, K)).astype(np.float16)
        w, s = marlin.pack_w8(to_dev(Q8), to_dev(S), G)
        call = lambda Ad, ws: marlin.gemm_w8(Ad, w, s, K, N, G, ws)
        ref = lambda M: w8_ref.gemm_w8(np.ascontiguousarray(A[:M]), Q8, S, Gn)
    else:
        case = inputs.make_dense(max_rows, K, N, G, seed=seed)
        w, s = marlin.pack(to_dev(case.q_kpacked), to_dev(case.S), G)
        A = case.A
        if fmt == "zp":
            Z = np.random.default_rng(seed + 1).integers(0, 16, size=case.S.shape, dtype=np.uint8)
            z = marlin.pack_zeros(to_dev(Z), K, N, G)
            call = lambda Ad, ws: marlin.gemm_zp(Ad, w, s, z, K, N, G, ws)
            ref = lambda M: zp_ref.gemm_zp(np.ascontiguousarray(A[:M]), case.q_kpacked, case.S, Z, case.G)
        else:
            call = lambda Ad, ws: marlin.gemm(Ad, w, s, K, N, G, ws)
            ref = lambda M: oracle_lib.gemm(np.ascontiguousarray(A[:M]), case.q_kpacked, case.S, case.G)
    return call, ref, to_dev(A), (K, N), what


@pytest.mark.parametrize("seed", [21, 22])
def test_random_chains_on_one_shared_workspace(oracle_lib, seed):
    # the deployment pattern: the layers of a model called in turn on one stream, each call sized for its own batch,
    # one workspace of the largest requirement shared by all of them, no synchronisation between the calls
    import torch
    import paper_2408_11743_b200 as marlin
    rng = np.random.default_rng(seed)
    rows = [1, 3, 8, 13, 16, 17, 32, 50, 64, 100, 128, 200, 300]
    for chain in range(12):
        layers = [_random_layer(rng, marlin, oracle_lib, 300) for _ in range(int(rng.integers(2, 5)))]
        calls = [(int(rng.integers(0, len(layers))), int(rng.choice(rows))) for _ in range(int(rng.integers(8, 20)))]
        need = max(marlin.workspace_bytes(M, *layers[li][3]) for li, M in calls)
        ws = torch.zeros(need, dtype=torch.uint8, device="cuda")
        outs = [layers[li][0](layers[li][2][:M], ws) for li, M in calls]
        torch.cuda.synchronize()
        assert marlin.read_status(ws) == 0
        refs = {}
        for i, ((li, M), C) in enumerate(zip(calls, outs)):
            if (li, M) not in refs:
                refs[(li, M)] = layers[li][1](M)
            bad, worst, _ = oracle_lib.check_tolerance(to_host(C), refs[(li, M)])
            assert bad == 0, (chain, i, layers[li][4], M, [(layers[a][4], m) for a, m in calls[max(0, i - 2):i]], worst)
        assert bool((ws[256:8192] == 0).all())
