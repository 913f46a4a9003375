"""GPU: marlin_pack / marlin_unpack are bit-exact (round trip, and equal to the CPU restatement of
the documented layout)."""
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


@pytest.mark.parametrize("K,N,G", [(128, 64, 128), (256, 192, 128), (512, 320, 256), (1024, 1024, 1024),
                                   (4096, 4096, 128), (11008, 4096, 128), (4096, 22016, -1),
                                   (256, 256, 64), (1024, 768, 32), (4096, 4096, 64)])
def test_pack_matches_layout_reference_and_round_trips(marlin, oracle_lib, K, N, G):
    from oracle import layout_ref
    case = inputs.make_dense(1, K, N, G, seed=K + N)
    Gn = case.G
    w, s = marlin.pack(to_dev(case.q_kpacked), to_dev(case.S), G)
    Q = oracle_lib.unpack_q(case.q_kpacked)
    want_w = layout_ref.pack_dense_weights(Q)
    want_s = layout_ref.pack_scales(case.S, sub=max(1, 128 // Gn))
    assert np.array_equal(to_host(w).view(np.uint32), want_w)
    assert np.array_equal(to_host(s).view(np.uint16), want_s.view(np.uint16).reshape(-1))
    q2, s2 = marlin.unpack(w, s, K, N, G)
    assert np.array_equal(to_host(q2).view(np.uint32), case.q_kpacked)
    assert np.array_equal(to_host(s2).view(np.uint16), case.S.view(np.uint16))
    assert s2.shape == (K // Gn, N)


def test_pack_every_nibble_pattern_in_every_position(marlin, oracle_lib):
    K, N = 256, 128
    k = np.arange(K)[:, None]
    n = np.arange(N)[None, :]
    for shift in range(16):
        Q = ((k * 7 + n * 3 + shift) % 16).astype(np.uint8)
        q = inputs.kpack(Q)
        S = np.ones((K // 128, N), dtype=np.float16)
        w, s = marlin.pack(to_dev(q), to_dev(S), 128)
        q2, _ = marlin.unpack(w, s, K, N, 128)
        assert np.array_equal(to_host(q2).view(np.uint32), q)


def test_pack_rejects_bad_arguments(marlin):
    import torch
    q = torch.zeros((16, 100), dtype=torch.int32, device="cuda")  # N = 100 is not a multiple of 64
    s = torch.ones((1, 100), dtype=torch.float16, device="cuda")
    with pytest.raises(marlin.MarlinError) as e:
        marlin.pack(q, s, 128)
    assert e.value.status == 2
    q = torch.zeros((32, 128), dtype=torch.int32, device="cuda")  # K = 256
    s = torch.ones((4, 128), dtype=torch.float16, device="cuda")
    with pytest.raises(marlin.MarlinError) as e:
        marlin.pack(q, s, 64)  # groups of 64 rows need N to be a multiple of 256
    assert e.value.status == 3
    q = torch.zeros((32, 256), dtype=torch.int32, device="cuda")
    for bad_g in (16, 48, 96, 100):  # neither 32, 64, a multiple of 128 nor K
        s = torch.ones((max(1, 256 // bad_g), 256), dtype=torch.float16, device="cuda")
        with pytest.raises(marlin.MarlinError) as e:
            marlin.pack(q, s, bad_g)
        assert e.value.status == 3
