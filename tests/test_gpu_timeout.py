"""GPU: the bounded waits inside the kernels really expire, report, and leave the device usable.

Nothing is faulted, trapped or hung here.  A TEST BUILD of the library (never the product .so) is compiled with
the wait limit shortened to a few milliseconds and with a hook that makes one CTA leave out the copies of one
pipeline stage when a magic word sits in the workspace.  The waits on that stage then run into their limit: the
CTA must set the abort flag and the status word MARLIN_ERR_DEVICE_TIMEOUT with a record of who waited on what,
every warp must run to the end of the kernel through its normal control flow (the call returns, the stream
synchronises), and an ordinary call afterwards, on a zeroed workspace, must be correct.
"""
import ctypes
import os

import numpy as np
import pytest

from paper_2408_11743_b200 import inputs
from gpu_util import to_dev, to_host

pytestmark = pytest.mark.gpu

WITHHOLD_MAGIC = 0x57495448


@pytest.fixture(scope="module")
def marlin():
    import torch
    assert torch.cuda.is_available()
    import paper_2408_11743_b200 as m
    m.lib()
    return m


@pytest.fixture(scope="module")
def test_lib(tmp_path_factory):
    from paper_2408_11743_b200 import build
    out = str(tmp_path_factory.mktemp("marlin_test_build") / "libmarlin_b200_testhooks.so")
    build.build(extra_flags=["-DMARLIN_TEST_HOOKS", "-DMARLIN_WAIT_LIMIT_NS=5000000ull"], out=out)
    L = ctypes.CDLL(out)
    vp, i, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
    L.marlin_gemm.argtypes = [vp, vp, vp, vp, i, i, i, i, vp, sz, vp]
    L.marlin_gemm.restype = i
    L.marlin_read_status.argtypes = [vp, vp]
    L.marlin_read_status.restype = i
    return L


@pytest.mark.parametrize("M,K,N", [(8, 4096, 4096), (64, 4096, 4096)])  # the warp-level kernel, the tcgen05 kernel
def test_an_expired_wait_is_reported_and_the_next_call_is_correct(marlin, test_lib, oracle_lib, M, K, N):
    import torch
    G = 128
    case = inputs.make_dense(M, K, N, G, seed=77 + M)
    w, s = marlin.pack(to_dev(case.q_kpacked), to_dev(case.S), G)   # the packed layout is the product's
    A = to_dev(case.A)
    C = torch.zeros((M, N), dtype=torch.float16, device="cuda")
    ws = marlin.new_workspace(M, K, N)
    stream = torch.cuda.current_stream().cuda_stream

    def call():
        return test_lib.marlin_gemm(A.data_ptr(), w.data_ptr(), s.data_ptr(), C.data_ptr(), M, K, N, G,
                                    ws.data_ptr(), ws.numel(), stream)

    # 1. an ordinary call of the test build works like the product
    assert call() == 0
    assert test_lib.marlin_read_status(ws.data_ptr(), stream) == 0
    ref = oracle_lib.gemm(case.A, case.q_kpacked, case.S, case.G)
    assert oracle_lib.check_tolerance(to_host(C), ref)[0] == 0

    # 2. the hook: worker 0 leaves out one stage; its waits expire after 5 ms instead of hanging
    ws.view(torch.int32)[7] = WITHHOLD_MAGIC
    assert call() == 0                        # the launch itself succeeds
    torch.cuda.synchronize()                  # ... and the kernel returns through its normal control flow
    assert test_lib.marlin_read_status(ws.data_ptr(), stream) == 8   # MARLIN_ERR_DEVICE_TIMEOUT
    rec = to_host(ws[:32]).view(np.int32)
    assert rec[0] == 8 and rec[1] == 0        # status word; the CTA that gave up is worker 0
    assert 0 <= rec[2] < 1024 and rec[5] > 0  # which thread waited, and that it polled before giving up
    assert rec[6] >= 4000                     # it waited the limit (in units of 1.024 us), not for ever

    # 3. the context is intact: zero the workspace (as after allocation) and call again
    ws.zero_()
    C.fill_(float("nan"))
    assert call() == 0
    assert test_lib.marlin_read_status(ws.data_ptr(), stream) == 0
    assert oracle_lib.check_tolerance(to_host(C), ref)[0] == 0
    # ... and so is the product library on the same device
    ws2 = marlin.new_workspace(M, K, N)
    C2 = to_host(marlin.gemm(A, w, s, K, N, G, ws2))
    assert marlin.read_status(ws2) == 0
    assert oracle_lib.check_tolerance(C2, ref)[0] == 0
