"""Helpers of the GPU parity tests: host arrays <-> device tensors, calls through the C ABI."""
import numpy as np


def to_dev(a: np.ndarray):
    import torch
    if a.dtype == np.uint32:
        a = a.view(np.int32)
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def to_host(t, dtype=None) -> np.ndarray:
    a = t.detach().cpu().numpy()
    if dtype is not None:
        a = a.view(dtype)
    return a


class DenseLayer:
    """A packed dense layer resident on the GPU, built through marlin_pack."""

    def __init__(self, marlin, q_kpacked: np.ndarray, S: np.ndarray, G: int, max_M: int = 128):
        self.m = marlin
        self.K, self.N, self.G = q_kpacked.shape[0] * 8, q_kpacked.shape[1], G
        self.w, self.s = marlin.pack(to_dev(q_kpacked), to_dev(S), G)
        self.ws = marlin.new_workspace(max_M, self.K, self.N)

    def __call__(self, A: np.ndarray) -> np.ndarray:
        import torch
        out = self.m.gemm(to_dev(A), self.w, self.s, self.K, self.N, self.G, self.ws)
        torch.cuda.synchronize()
        assert self.m.read_status(self.ws) == 0
        return to_host(out)


class SparseLayer:
    """A packed 2:4 layer resident on the GPU, built through marlin_pack_sparse24 from a generated case."""

    def __init__(self, marlin, case, max_M):
        self.m, self.K, self.N, self.G = marlin, case.K, case.N, case.G
        self.w, self.meta, self.s = marlin.pack_sparse24(to_dev(case.qc_kpacked), to_dev(case.idx), to_dev(case.S), case.G)
        self.ws = marlin.new_workspace(max_M, self.K, self.N)

    def __call__(self, A):
        import torch
        out = self.m.gemm_sparse24(to_dev(A), self.w, self.meta, self.s, self.K, self.N, self.G, self.ws)
        torch.cuda.synchronize()
        assert self.m.read_status(self.ws) == 0
        return to_host(out)
