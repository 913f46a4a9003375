"""GPU: the entry point with the built-in workspace gives what marlin_gemm gives.

marlin_gemm_static_ws exists for callers that cannot allocate device memory (a plug-in inside a
pre-planned execution graph, a runtime that forbids cudaMalloc after start-up): its scratch memory
is a fixed array inside the library.  This file is collected last on purpose, so that a run that
stops at the first failure has already run every other test; it also passes when run alone.

The cases are chosen so that the kernels really use the array: the partial tiles and arrival counters
of the fix-up across CTAs live in it whenever a column tile is shared by CTAs that are not one
thread-block cluster (forced here through the library's tuning switches, and true by itself of the
shapes with more CTAs per tile than a cluster holds or with even stripes).
"""
import ctypes

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


CASES = [
    # (M, K, N, G, environment): all of them reduce partial tiles through the workspace
    (16, 4096, 4096, 128, {"MARLIN_B200_CLUSTER": "0"}),
    (5, 2048, 1536, -1, {"MARLIN_B200_CLUSTER": "0"}),
    (16, 8192, 1024, 128, {}),      # many CTAs per column tile
    (8, 4096, 22016, 128, {}),      # even stripes, segments in the middle of a stripe
    (3, 1024, 192, 128, {"MARLIN_B200_SPLIT": "0"}),
]


@pytest.mark.parametrize("M,K,N,G,env", CASES)
def test_static_workspace_entry_matches_marlin_gemm_twice_in_a_row(marlin, oracle_lib, monkeypatch, M, K, N, G, env):
    import torch
    for k, v in env.items():
        monkeypatch.setenv(k, v)
    case = inputs.make_dense(M, K, N, G, seed=4242 + M)
    w, s = marlin.pack(to_dev(case.q_kpacked), to_dev(case.S), G)
    A = to_dev(case.A)
    ws = marlin.new_workspace(M, K, N)
    want = to_host(marlin.gemm(A, w, s, K, N, G, ws))
    torch.cuda.synchronize()
    # a plain call of another shape in between, on the same stream, with a workspace of its own
    other = inputs.make_dense(7, 512, 320, 128, seed=99)
    ow, os_ = marlin.pack(to_dev(other.q_kpacked), to_dev(other.S), 128)
    ows = marlin.new_workspace(7, 512, 320)
    out = torch.empty((M, N), dtype=torch.float16, device="cuda")
    for call in range(3):
        out.fill_(float("nan"))  # every element must be rewritten by the call
        if call == 2:
            marlin.gemm(to_dev(other.A), ow, os_, 512, 320, 128, ows)
        marlin.gemm_static_ws(A, w, s, K, N, G, out=out)
        torch.cuda.synchronize()
        got = to_host(out)
        bad, worst, _ = oracle_lib.check_tolerance(got, want)  # the bound the other parity tests use
        assert bad == 0, f"call {call}: {bad} elements differ (worst error/allowance {worst:.3f})"
        assert np.array_equal(got.view(np.uint16), want.view(np.uint16))  # same kernels, same order: same bits
    # and against the oracle itself
    bad, worst, _ = oracle_lib.check_tolerance(got, oracle_lib.gemm(case.A, case.q_kpacked, case.S, case.G))
    assert bad == 0, worst


def test_static_workspace_entry_checks_its_arguments_before_queueing(marlin):
    from paper_2408_11743_b200 import binding
    K, N = 256, 128
    case = inputs.make_dense(binding.STATIC_WS_MAX_M + 1, K, N, 128, seed=1)
    w, s = marlin.pack(to_dev(case.q_kpacked), to_dev(case.S), 128)
    with pytest.raises(marlin.MarlinError) as e:
        marlin.gemm_static_ws(to_dev(case.A), w, s, K, N, 128)
    assert e.value.status == 2
    L = marlin.lib()
    fake, odd = ctypes.c_void_p(0x1000), ctypes.c_void_p(0x1008)  # never dereferenced: the checks fail first
    assert L.marlin_gemm_static_ws(None, fake, fake, fake, 1, K, N, 128, None) == 1
    assert L.marlin_gemm_static_ws(fake, fake, fake, fake, 1, K + 1, N, 128, None) == 2
    assert L.marlin_gemm_static_ws(fake, fake, fake, fake, 1, K, N, 96, None) == 3
    assert L.marlin_gemm_static_ws(odd, fake, fake, fake, 1, K, N, 128, None) == 4
