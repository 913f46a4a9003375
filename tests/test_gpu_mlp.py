"""The gated MLP chain (marlin_interleave_gate_up, marlin_gemm_swiglu, marlin_mlp_swiglu) against the CPU oracle.

H is compared with a bound derived from the layer's: the products g, u may be off by t(x) = 5e-3 (|x| + rms), the
activation has slope below 1.1, so |H - H_ref| <= 1.1 |u| t(g) + |silu(g)| t(u) + t(g) t(u) + two fp16 roundings.  The
down projection is compared with the layer oracle applied to the H the GPU produced (its inputs are then identical).
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


def _mlp_case(M, K, I, N, G, seed):
    gate = inputs.make_dense(M, K, I, G, seed=seed)
    up = inputs.make_dense(M, K, I, G, seed=seed + 1)
    down = inputs.make_dense(M, I, N, G, seed=seed + 2)
    return gate, up, down


def _h_bound(g, u, H_ref):
    g64, u64 = g.astype(np.float64), u.astype(np.float64)
    both = np.concatenate([g64.ravel(), u64.ravel()])
    rms = float(np.sqrt(np.mean(both ** 2)))
    tg, tu = 5e-3 * (np.abs(g64) + rms), 5e-3 * (np.abs(u64) + rms)
    from oracle import mlp_ref
    return 1.1 * np.abs(u64) * tg + np.abs(mlp_ref.silu(g64)) * tu + tg * tu + 2.0 ** -9 * np.abs(H_ref.astype(np.float64)) + 1e-7


def test_interleave_matches_the_definition(marlin):
    import torch
    from oracle import mlp_ref
    gate, up, _ = _mlp_case(1, 256, 96, 64, 128, seed=1)
    q, s = marlin.interleave_gate_up(to_dev(gate.q_kpacked), to_dev(gate.S), to_dev(up.q_kpacked), to_dev(up.S), 128)
    torch.cuda.synchronize()
    assert np.array_equal(to_host(q).view(np.uint32), mlp_ref.interleave(gate.q_kpacked, up.q_kpacked))
    assert np.array_equal(to_host(s), mlp_ref.interleave(gate.S, up.S))


# I chosen so that the fused layer (2 I columns) lands on every kernel: multiples of 256, of 128 only, of 64 only
@pytest.mark.parametrize("M,K,I,G", [(1, 1024, 256, 128), (8, 2048, 512, 128), (16, 1024, 96, 128), (16, 1024, 160, -1),
                                     (17, 1024, 256, 128), (40, 2048, 384, 128), (64, 1024, 192, 128), (128, 1024, 512, 128),
                                     (33, 1024, 160, 128), (300, 1024, 256, 128), (5, 4096, 11008, 128)])
def test_fused_activation_matches_the_oracle(marlin, oracle_lib, M, K, I, G):
    import torch
    from oracle import mlp_ref
    gate, up, _ = _mlp_case(M, K, I, 64, G, seed=M + K + I)
    A = gate.A
    q, s = marlin.interleave_gate_up(to_dev(gate.q_kpacked), to_dev(gate.S), to_dev(up.q_kpacked), to_dev(up.S), G)
    w_packed, s_packed = marlin.pack(q, s, G)
    ws = marlin.new_workspace(M, K, 2 * I)
    H = to_host(marlin.gemm_swiglu(to_dev(A), w_packed, s_packed, K, 2 * I, G, ws))
    torch.cuda.synchronize()
    assert marlin.read_status(ws) == 0
    g, u, H_ref = mlp_ref.gate_up(A, gate.q_kpacked, gate.S, up.q_kpacked, up.S, gate.G)
    err = np.abs(H.astype(np.float64) - H_ref.astype(np.float64))
    bound = _h_bound(g, u, H_ref)
    assert np.all(err <= bound), f"worst ratio {np.max(err / bound):.3f}"
    assert np.all(to_host(ws)[256:8192] == 0)


@pytest.mark.parametrize("M,K,I,N,G", [(1, 1024, 256, 512, 128), (16, 2048, 512, 1024, 128), (48, 1024, 384, 256, 128),
                                       (200, 1024, 256, 512, 128), (4, 4096, 11008, 4096, 128)])
def test_two_launch_chain(marlin, oracle_lib, M, K, I, N, G):
    import torch
    from oracle import mlp_ref
    gate, up, down = _mlp_case(M, K, I, N, G, seed=7 * M + I)
    A = gate.A
    q, s = marlin.interleave_gate_up(to_dev(gate.q_kpacked), to_dev(gate.S), to_dev(up.q_kpacked), to_dev(up.S), G)
    w_gu, s_gu = marlin.pack(q, s, G)
    w_d, s_d = marlin.pack(to_dev(down.q_kpacked), to_dev(down.S), G)
    ws = marlin.new_workspace(M, max(K, I), max(2 * I, N))
    need = max(marlin.workspace_bytes(M, K, 2 * I), marlin.workspace_bytes(M, I, N))
    if ws.numel() < need:
        ws = torch.zeros(need, dtype=torch.uint8, device="cuda")
    H = torch.empty((M, I), dtype=torch.float16, device="cuda")
    for _ in range(3):  # the chain several times over on one workspace: the launches overlap at their edges
        C = marlin.mlp_swiglu(to_dev(A), w_gu, s_gu, w_d, s_d, K, I, N, G, ws, H=H)
    torch.cuda.synchronize()
    assert marlin.read_status(ws) == 0
    Hh = to_host(H)
    g, u, H_ref = mlp_ref.gate_up(A, gate.q_kpacked, gate.S, up.q_kpacked, up.S, gate.G)
    err = np.abs(Hh.astype(np.float64) - H_ref.astype(np.float64))
    assert np.all(err <= _h_bound(g, u, H_ref))
    if I * N <= 1 << 22:
        C_ref = oracle_lib.gemm(Hh, down.q_kpacked, down.S, down.G)
        bad, worst, _ = oracle_lib.check_tolerance(to_host(C), C_ref)
    else:
        rng = np.random.default_rng(0)
        ms, ns = rng.integers(0, M, 2048), rng.integers(0, N, 2048)
        ref = oracle_lib.gemm_samples(Hh, down.q_kpacked, down.S, down.G, ms, ns)
        bad, worst, _ = oracle_lib.check_tolerance(np.ascontiguousarray(to_host(C)[ms, ns]), ref)
    assert bad == 0, worst
