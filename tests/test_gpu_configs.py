"""GPU parity on every case of the five workload configs, at full size, on sampled outputs.

Walks inputs.iter_cases(1..5): every layer shape, every batch size, both scale modes of config 4 and the 2:4
layer of config 5, each through the C ABI in the launch configuration the benchmark times.  The full product
of the largest layers would take the CPU oracle minutes, so each case is checked on 2048 outputs drawn at
random that the oracle computes one by one (oracle.gemm_samples); small cases are checked in full as well.

Bound: |C - C_ref| <= 5e-3 * (|C_ref| + rms(C_ref)), with rms taken over the SAMPLED outputs (2048 draws
estimate the rms of the full result to about two per cent).
"""
import numpy as np
import pytest

from paper_2408_11743_b200 import inputs
from gpu_util import to_dev, to_host

pytestmark = pytest.mark.gpu

N_SAMPLES = 2048


@pytest.fixture(scope="module")
def marlin():
    import torch
    assert torch.cuda.is_available()
    import paper_2408_11743_b200 as m
    m.lib()
    return m


def _check_samples(oracle_lib, C, A, q_kpacked, S, G, seed, what):
    M, N = C.shape
    rng = np.random.default_rng(seed)
    ms = rng.integers(0, M, N_SAMPLES)
    ns = rng.integers(0, N, N_SAMPLES)
    # every row and the first and last columns of the layer are among the samples
    ms[:M] = np.arange(M)[:N_SAMPLES]
    ns[0], ns[1] = 0, N - 1
    ref = oracle_lib.gemm_samples(A, q_kpacked, S, G, ms, ns)
    bad, worst, rms = oracle_lib.check_tolerance(np.ascontiguousarray(C[ms, ns]), ref)
    assert bad == 0, f"{what}: {bad} of {N_SAMPLES} sampled outputs out of tolerance (worst {worst:.3f}, sample rms {rms:.3f})"
    assert np.all(np.isfinite(C.astype(np.float32))), what


@pytest.mark.parametrize("config", [1, 2, 3, 4])
def test_every_dense_case_of_the_config_matches_the_oracle_on_sampled_outputs(marlin, oracle_lib, config):
    import torch
    for name, M, K, N, G, seed in inputs.iter_cases(config):
        case = inputs.make_dense(M, K, N, G, seed)
        w, s = marlin.pack(to_dev(case.q_kpacked), to_dev(case.S), G)
        ws = marlin.new_workspace(M, K, N)
        C = to_host(marlin.gemm(to_dev(case.A), w, s, K, N, G, ws))
        torch.cuda.synchronize()
        assert marlin.read_status(ws) == 0
        _check_samples(oracle_lib, C, case.A, case.q_kpacked, case.S, case.G, seed + 1,
                       f"config {config} {name} M={M} K={K} N={N} G={G}")
        del w, s, ws
        torch.cuda.empty_cache()


def test_every_sparse_case_of_config_5_matches_the_oracle_on_sampled_outputs(marlin, oracle_lib):
    import torch
    for name, M, K, N, G, seed in inputs.iter_cases(5):
        case = inputs.make_sparse24(M, K, N, G, seed)
        w, meta, s = marlin.pack_sparse24(to_dev(case.qc_kpacked), to_dev(case.idx), to_dev(case.S), G)
        ws = marlin.new_workspace(M, K, N)
        C = to_host(marlin.gemm_sparse24(to_dev(case.A), w, meta, s, K, N, G, ws))
        torch.cuda.synchronize()
        assert marlin.read_status(ws) == 0
        # the oracle's expansion: code 8 (value zero) at the pruned positions, then the dense definition
        q_dense = oracle_lib.pack_q(oracle_lib.sparse24_expand(case.qc_kpacked, case.idx))
        _check_samples(oracle_lib, C, case.A, q_dense, case.S, case.G, seed + 1, f"config 5 M={M}")
