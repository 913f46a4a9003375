"""Host-side checks that need no GPU: the library loads, exports every declared symbol, and its
size / planning arithmetic is right."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


@pytest.fixture(scope="module")
def marlin():
    from paper_2408_11743_b200 import build
    build.build()
    import paper_2408_11743_b200 as m
    return m


def test_library_exports_every_declared_symbol(marlin):
    header = open(os.path.join(ROOT, "include", "marlin_b200.h")).read()
    declared = re.findall(r"MARLIN_API\s+[\w\s\*]+?\b(marlin_\w+)\s*\(", header)
    assert len(declared) >= 13
    L = ctypes.CDLL(marlin.library_path())
    for name in declared:
        assert hasattr(L, name), name
    from paper_2408_11743_b200 import binding
    assert sorted(set(declared)) == sorted(binding.EXPORTS)


def test_missing_library_fails_loudly(monkeypatch, marlin):
    from paper_2408_11743_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "_LIB_PATH", "/nonexistent/libmarlin_b200.so")
    with pytest.raises(RuntimeError):
        binding.lib()


def test_size_queries(marlin):
    L = marlin.lib()
    assert L.marlin_packed_weight_bytes(4096, 4096, 0) == 4096 * 4096 // 2
    assert L.marlin_packed_weight_bytes(4096, 4096, 1) == 4096 * 4096 // 4
    assert L.marlin_packed_meta_bytes(4096, 4096) == 4096 * 4096 // 8
    assert L.marlin_packed_scale_bytes(4096, 4096, 128) == 2 * 32 * 4096
    assert L.marlin_packed_scale_bytes(4096, 4096, -1) == 2 * 4096
    assert L.marlin_packed_scale_bytes(4096, 4096, 4096) == 2 * 4096
    assert L.marlin_packed_scale_bytes(4096, 4096, 100) == 0     # not 32, 64, a multiple of 128 or K
    assert L.marlin_packed_scale_bytes(4096, 4096, 64) == 2 * 64 * 4096
    assert L.marlin_packed_scale_bytes(4096, 4096, 32) == 2 * 128 * 4096
    assert L.marlin_packed_scale_bytes(4096, 4160, 64) == 0      # groups of 64 rows need N % 256 == 0
    assert L.marlin_packed_scale_bytes(4096, 4096, 16) == 0
    assert L.marlin_packed_scale_bytes(4096, 4096, 384) == 0     # does not divide K
    assert L.marlin_packed_weight_bytes(4000, 4096, 0) == 0      # K % 128
    assert L.marlin_packed_weight_bytes(4096, 4000, 0) == 0      # N % 64
    assert L.marlin_workspace_bytes(0, 4096, 4096) == 0
    # the query covers dense and 2:4 layers of the shape: header, partial-tile slots, and the fp32 tiles of the tcgen05
    # kernel (which 2:4 layers use from one row on, dense ones from 17): constant up to 32 rows, then growing
    assert L.marlin_workspace_bytes(1, 4096, 4096) == L.marlin_workspace_bytes(16, 4096, 4096) \
        <= L.marlin_workspace_bytes(32, 4096, 4096) < L.marlin_workspace_bytes(64, 4096, 4096) \
        < L.marlin_workspace_bytes(128, 4096, 4096)
    assert L.marlin_status_string(0) == b"ok"
    assert L.marlin_status_string(8).startswith(b"bounded wait")


def test_argument_checks_return_before_any_cuda_call(marlin):
    L = marlin.lib()
    assert L.marlin_gemm(None, None, None, None, 1, 4096, 4096, 128, None, 0, None) == 1   # NULL
    fake = ctypes.c_void_p(0x1000)  # aligned, never dereferenced: every check below fails first
    assert L.marlin_gemm(fake, fake, fake, fake, 0, 4096, 4096, 128, fake, 1 << 30, None) == 2
    assert L.marlin_gemm(fake, fake, fake, fake, 1, 4097, 4096, 128, fake, 1 << 30, None) == 2
    assert L.marlin_gemm(fake, fake, fake, fake, 1, 4096, 4096, 96, fake, 1 << 30, None) == 3
    odd = ctypes.c_void_p(0x1008)
    assert L.marlin_gemm(odd, fake, fake, fake, 1, 4096, 4096, 128, fake, 1 << 30, None) == 4
    assert L.marlin_gemm(fake, fake, fake, fake, 1, 4096, 4096, 128, fake, 16, None) == 5
    assert L.marlin_pack(None, fake, fake, fake, 4096, 4096, 128, None) == 1
    assert L.marlin_pack(fake, fake, fake, fake, 4096, 4000, 128, None) == 2
    assert L.marlin_read_status(None, None) == 1


SHAPES = [(4096, 4096), (8192, 8192), (4096, 12288), (4096, 22016), (11008, 4096), (8192, 57344), (28672, 8192),
          (28672, 1024), (128, 64), (256, 192)]


@pytest.mark.parametrize("K,N", SHAPES)
@pytest.mark.parametrize("M", [1, 16, 32, 128])
@pytest.mark.parametrize("sms", [148, 132, 7])
def test_stripe_partition_covers_every_unit_once(marlin, K, N, M, sms):
    n_tile, workers, bounds = marlin.plan_stripes(M, K, N, sms)
    assert n_tile in (64, 128, 256) and N % n_tile == 0
    kb = K // 128
    units = (N // n_tile) * kb
    assert 1 <= workers <= min(sms, units)
    assert bounds[0] == 0 and bounds[-1] == units and len(bounds) == workers + 1
    sizes = [b - a for a, b in zip(bounds, bounds[1:])]
    assert min(sizes) >= 1                                           # contiguous, nobody idle
    if max(sizes) - min(sizes) <= 1 and workers == min(sms, units):
        # even stripes: the device finds the owner of unit x as floor(((x + 1) * P - 1) / U)
        import bisect
        step = max(1, units // 997)
        for x in list(range(0, units, step)) + [units - 1]:
            owner = ((x + 1) * workers - 1) // units
            assert bounds[owner] <= x < bounds[owner + 1]
            assert owner == bisect.bisect_right(bounds, x) - 1
    else:
        # tile-aligned form: the same number S of k-ranges in every column tile, none crossing a tile
        # boundary, their lengths within one k-block of each other
        ncols = N // n_tile
        assert workers % ncols == 0
        S = workers // ncols
        assert S <= kb
        for w in range(workers):
            assert bounds[w] // kb == (bounds[w + 1] - 1) // kb == w // S
        assert max(sizes) - min(sizes) <= 1


@pytest.mark.parametrize("K,N,tile,workers,form", [
    (8192, 8192, 128, 128, "aligned"),     # 64 tiles x 2 k-ranges of 32 stages: twelve consumer warps pay from 16 on
    (4096, 4096, 64, 128, "aligned"),      # 64 tiles x 2 k-ranges
    (4096, 12288, 256, 144, "aligned"),    # 48 tiles x 3 k-ranges
    (11008, 4096, 128, 128, "aligned"),    # 32 tiles x 4 k-ranges
    (2048, 8192, 64, 128, "aligned"),      # short K: one 64-column tile and all of K per CTA, no fix-up across CTAs
    (4096, 22016, 128, 148, "even"),       # 172 tiles do not divide 148 SMs: even stripes
    (28672, 8192, 128, 128, "aligned"),    # 64 tiles x 2 k-ranges of 112 stages (as fast as even stripes on 148 SMs)
    (8192, 28672, 128, 148, "even"),       # 224 tiles: idle SMs would cost more than the late finishers
])
def test_partition_chosen_for_the_layer_shapes_of_the_benchmarks(marlin, K, N, tile, workers, form):
    n_tile, w, bounds = marlin.plan_stripes(1, K, N, 148)
    assert (n_tile, w) == (tile, workers)
    kb = K // 128
    crosses = any(bounds[i] // kb != (bounds[i + 1] - 1) // kb for i in range(w))
    assert crosses == (form == "even")


def test_byte_model_matches_paper():
    from paper_2408_11743_b200 import roofline
    rows = [l.split() for l in open(os.path.join(GOLDEN, "byte_model.txt")) if l.strip() and l[0] != "#"]
    for M, K, N, bits, macs in [tuple(map(int, r)) for r in rows[:-1]]:
        assert roofline.algorithmic_bytes(M, K, N, K, scales=False) * 8 == bits
        assert roofline.flops(M, K, N) == 2 * macs
    ideal = float(rows[-1][0])
    # 16 / 4.125 = 3.8788; the paper prints it cut to two decimals
    assert int(100 * roofline.weight_bits_fp16() / roofline.weight_bits_w4(128)) / 100 == ideal
    # with scales: 2 bytes per (group, column)
    assert roofline.weight_bytes(8192, 8192, 128) == 8192 * 8192 // 2 + 2 * 64 * 8192
    assert roofline.weight_bytes(8192, 8192, 128, sparse24=True) == 8192 * 8192 // 4 + 8192 * 8192 // 8 + 2 * 64 * 8192


def test_no_kernel_of_the_built_library_spills_registers_to_memory():
    # the register allocator's report of the last build: a kernel that starts spilling hundreds of bytes has lost its
    # place in the register file (seen once: an epilogue variant cost the large-batch kernel a third of its speed)
    from paper_2408_11743_b200 import build
    build.build()
    report = build.spill_report()
    if not report:
        build.build(force=True)
        report = build.spill_report()
    assert report, "no ptxas report beside the library"
    assert len(report) >= 20
    bad = {k: v for k, v in report.items() if v[1] > 64}
    assert not bad, bad
