"""GPU: the entry point with the built-in workspace gives what marlin_gemm gives.

marlin_gemm_static_ws exists for callers that cannot allocate device memory (a plug-in inside a
pre-planned execution graph, a runtime that forbids cudaMalloc after start-up): its scratch memory
is a fixed array inside the library.  This file is collected last on purpose, so that a run that
stops at the first failure has already run every other test; it also passes when run alone.
"""
import numpy as np
import pytest

from paper_2408_11743_b200 import inputs
from gpu_util import to_dev, to_host

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def marlin():
    import torch
    assert torch.cuda.is_available()
    import paper_2408_11743_b200 as m
    m.lib()
    return m


@pytest.mark.parametrize("M,K,N,G", [(16, 4096, 4096, 128), (5, 2048, 1536, -1)])
def test_static_workspace_entry_matches_marlin_gemm_twice_in_a_row(marlin, oracle_lib, M, K, N, G):
    import torch
    case = inputs.make_dense(M, K, N, G, seed=4242 + M)
    w, s = marlin.pack(to_dev(case.q_kpacked), to_dev(case.S), G)
    A = to_dev(case.A)
    ws = marlin.new_workspace(M, K, N)
    want = to_host(marlin.gemm(A, w, s, K, N, G, ws))
    torch.cuda.synchronize()
    out = torch.empty((M, N), dtype=torch.float16, device="cuda")
    for call in range(2):
        out.fill_(float("nan"))  # every element must be rewritten by the call
        marlin.gemm_static_ws(A, w, s, K, N, G, out=out)
        torch.cuda.synchronize()
        got = to_host(out)
        bad, worst, _ = oracle_lib.check_tolerance(got, want)  # the bound the other parity tests use
        assert bad == 0, f"call {call}: {bad} elements differ (worst error/allowance {worst:.3f})"
        assert np.array_equal(got.view(np.uint16), want.view(np.uint16))  # same kernels, same order: same bits
    # and against the oracle itself
    bad, worst, _ = oracle_lib.check_tolerance(got, oracle_lib.gemm(case.A, case.q_kpacked, case.S, case.G))
    assert bad == 0, worst


def test_static_workspace_entry_rejects_large_batches(marlin):
    import torch
    from paper_2408_11743_b200 import binding
    K, N = 256, 128
    case = inputs.make_dense(binding.STATIC_WS_MAX_M + 1, K, N, 128, seed=1)
    w, s = marlin.pack(to_dev(case.q_kpacked), to_dev(case.S), 128)
    with pytest.raises(marlin.MarlinError) as e:
        marlin.gemm_static_ws(to_dev(case.A), w, s, K, N, 128)
    assert e.value.status == 2
