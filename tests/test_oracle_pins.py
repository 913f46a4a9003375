"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these tests retypes the oracle's own formula in floating point: they use
integer or exact rational arithmetic, brute-force search over all fp16 values,
numpy's library routines on special cases, closed forms, and the worked example
of the paper (tests/golden/dequant_magic.txt).
"""
import bisect
import os
from fractions import Fraction

import numpy as np
import pytest

from paper_2408_11743_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ---------- exact helpers, independent of the oracle -------------------------------------------

def _f16_fraction(bits: int) -> Fraction:
    s = -1 if bits >> 15 else 1
    e = (bits >> 10) & 31
    f = bits & 1023
    assert e != 31
    if e == 0:
        return s * Fraction(f, 1 << 24)
    return s * Fraction(1024 + f, 1024) * (Fraction(2) ** (e - 15))


_POS = [(_f16_fraction(b), b) for b in range(0x7C00)]  # ascending, finite non-negative halves
_POS_VALS = [v for v, _ in _POS]


def _round_fraction_to_f16_bits(x: Fraction) -> int:
    """Nearest fp16 by search over every finite half; ties to the even bit pattern; overflow to inf."""
    sign = 0x8000 if x < 0 else 0
    a = abs(x)
    top = _POS_VALS[-1]
    if a >= top + (Fraction(2) ** 4):  # beyond the midpoint between 65504 and 65536 (tie goes to inf = even)
        return sign | 0x7C00
    i = bisect.bisect_left(_POS_VALS, a)
    if i == len(_POS_VALS):
        return sign | _POS[-1][1]
    if _POS_VALS[i] == a or i == 0:
        return sign | _POS[i][1]
    lo, hi = _POS[i - 1], _POS[i]
    dl, dh = a - lo[0], hi[0] - a
    if dl < dh:
        return sign | lo[1]
    if dh < dl:
        return sign | hi[1]
    return sign | (lo[1] if lo[1] % 2 == 0 else hi[1])


def _exact_reference(A, Q, S, G):
    """C by exact rational arithmetic, rounded by exhaustive search (tiny shapes only)."""
    M, K = A.shape
    N = Q.shape[1]
    Ab = A.view(np.uint16)
    Sb = S.view(np.uint16)
    out = np.empty((M, N), dtype=np.uint16)
    for m in range(M):
        for n in range(N):
            acc = Fraction(0)
            for k in range(K - 1, -1, -1):  # a different order from the oracle's: the sum is exact anyway
                acc += _f16_fraction(int(Ab[m, k])) * (int(Q[k, n]) - 8) * _f16_fraction(int(Sb[k // G, n]))
            out[m, n] = _round_fraction_to_f16_bits(acc)
    return out.view(np.float16)


# ---------- P4: the rounding routine --------------------------------------------------------------

def test_f16_roundtrip_all_bit_patterns(oracle_lib):
    bits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    h = bits.view(np.float16)
    d = oracle_lib.f16_to_f64(h)
    finite = np.isfinite(h)
    assert np.array_equal(d[finite], h[finite].astype(np.float64))  # numpy's widening is exact
    assert np.all(np.isnan(d[np.isnan(h)]))
    back = oracle_lib.f64_to_f16(d).view(np.uint16)
    notnan = ~np.isnan(h)
    assert np.array_equal(back[notnan], bits[notnan])
    assert np.all(np.isnan(back[~notnan].view(np.float16)))


def test_f16_midpoints_tie_to_even(oracle_lib):
    # exact midpoint of every pair of neighbouring non-negative halves (the pair max-finite/inf included)
    lo = np.arange(0, 0x7C00, dtype=np.uint16)
    a = lo.view(np.float16).astype(np.float64)
    b = np.concatenate([a[1:], [65536.0]])
    mid = (a + b) / 2  # exact in fp64
    got = oracle_lib.f64_to_f16(mid).view(np.uint16)
    want = np.where(lo % 2 == 0, lo, lo + 1).astype(np.uint16)
    assert np.array_equal(got, want)
    gotneg = oracle_lib.f64_to_f16(-mid).view(np.uint16)
    assert np.array_equal(gotneg, want | 0x8000)
    # one fp64 ulp to either side of a midpoint must leave the tie
    up = np.nextafter(mid, np.inf)
    dn = np.nextafter(mid, -np.inf)
    assert np.array_equal(oracle_lib.f64_to_f16(up).view(np.uint16), (lo + 1).astype(np.uint16))
    assert np.array_equal(oracle_lib.f64_to_f16(dn[1:]).view(np.uint16), lo[1:])


def test_f16_rounding_matches_numpy_on_random_doubles(oracle_lib):
    rng = np.random.default_rng(7)
    x = np.concatenate([
        rng.standard_normal(400000) * 10.0 ** rng.integers(-9, 6, 400000),
        rng.uniform(-70000, 70000, 200000),
        rng.uniform(-1e-4, 1e-4, 200000),
        np.array([0.0, -0.0, np.inf, -np.inf, 65504.0, 65519.999, 65520.0, 65520.001, 2.0 ** -24, 2.0 ** -25,
                  np.nextafter(2.0 ** -25, 1), 1e-300, -1e300]),
    ])
    with np.errstate(over="ignore"):
        want = x.astype(np.float16).view(np.uint16)
    got = oracle_lib.f64_to_f16(x).view(np.uint16)
    assert np.array_equal(got, want)


# ---------- P1: canonical packing -----------------------------------------------------------------

def test_kpack_roundtrip_and_nibble_order(oracle_lib):
    rng = np.random.default_rng(3)
    Q = rng.integers(0, 16, size=(64, 24), dtype=np.uint8)
    w = oracle_lib.pack_q(Q)
    assert np.array_equal(oracle_lib.unpack_q(w), Q)
    assert np.array_equal(inputs.kpack(Q), w)  # the input generator and the oracle agree on the format
    # nibble j of word (kb, n) is row 8*kb + j: one marked row at a time
    for k in (0, 1, 7, 8, 13, 63):
        Z = np.zeros((64, 3), dtype=np.uint8)
        Z[k, 1] = 0xF
        wz = oracle_lib.pack_q(Z)
        assert wz[k // 8, 1] == np.uint32(0xF) << np.uint32(4 * (k % 8))
        assert int(wz.astype(np.uint64).sum()) == int(wz[k // 8, 1])
    # every nibble pattern in every position
    allpat = np.arange(16, dtype=np.uint8).repeat(8)[:, None] * np.ones((1, 2), dtype=np.uint8)
    assert np.array_equal(oracle_lib.unpack_q(oracle_lib.pack_q(allpat)), allpat)


# ---------- P2 / P3: dequantisation -----------------------------------------------------------------

def test_dequant_exact_for_every_code_and_finite_scale(oracle_lib):
    bits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    h = bits.view(np.float16)
    fin = bits[np.isfinite(h)]
    S = fin.view(np.float16)[None, :]
    # integer decomposition of the scale: s = sgn * mant * 2^ex
    e = ((fin >> 10) & 31).astype(np.int64)
    f = (fin & 1023).astype(np.int64)
    mant = np.where(e == 0, f, 1024 + f)
    ex = np.where(e == 0, -24, e - 25)
    sgn = np.where(fin >> 15, -1, 1).astype(np.int64)
    for q in range(16):
        Q = np.full((1, fin.size), q, dtype=np.uint8)
        W = oracle_lib.dequant(Q, S, 1)[0]
        # W / 2^ex must be exactly the integer (q - 8) * sgn * mant
        scaled = np.ldexp(W, -ex.astype(np.int32))
        assert np.array_equal(scaled, ((q - 8) * sgn * mant).astype(np.float64))


def test_dequant_matches_paper_worked_example(oracle_lib):
    rows = [l.split() for l in open(os.path.join(GOLDEN, "dequant_magic.txt")) if l.strip() and l[0] != "#"]
    assert len(rows) == 16
    one = np.ones((1, 1), dtype=np.float16)
    for code, blo, vlo, bhi, vhi, signed in rows:
        code, vlo, vhi, signed = int(code), int(vlo), int(vhi), int(signed)
        lo = np.array([int(blo, 16)], dtype=np.uint16).view(np.float16)[0]
        hi = np.array([int(bhi, 16)], dtype=np.uint16).view(np.float16)[0]
        assert int(blo, 16) == (0x6400 | code) and int(bhi, 16) == (0x6400 | (code << 4))
        assert float(lo) == vlo and float(hi) == vhi
        # the paper's conversion, in fp16 arithmetic
        m1032 = np.array([0x6408], dtype=np.uint16).view(np.float16)[0]
        assert float(np.float16(lo - m1032)) == signed
        sixteenth = np.array([0x2C00], dtype=np.uint16).view(np.float16)[0]
        m72 = np.array([0xD480], dtype=np.uint16).view(np.float16)[0]
        assert float(np.float16(np.float32(hi) * np.float32(sixteenth) + np.float32(m72))) == signed
        # ... gives what the oracle calls the value of that code at scale 1
        W = oracle_lib.dequant(np.array([[code]], dtype=np.uint8), one, 1)
        assert W[0, 0] == signed


# ---------- P8: brute force in exact arithmetic ----------------------------------------------------

@pytest.mark.parametrize("M,K,N,G,seed", [(1, 16, 3, 16, 0), (3, 32, 5, 8, 1), (2, 64, 4, 32, 2), (5, 48, 2, 16, 3)])
def test_gemm_equals_exact_rational_result(oracle_lib, M, K, N, G, seed):
    case = inputs.make_dense(M, K, N, G, seed)
    Q = oracle_lib.unpack_q(case.q_kpacked)
    want = _exact_reference(case.A, Q, case.S, G)
    got = oracle_lib.gemm(case.A, case.q_kpacked, case.S, G)
    assert np.array_equal(got.view(np.uint16), want.view(np.uint16))


def test_gemm_exact_with_wide_dynamic_range(oracle_lib):
    # large and tiny activations and scales, results near overflow and in the subnormal range
    rng = np.random.default_rng(11)
    M, K, N, G = 4, 32, 6, 16
    A = (rng.standard_normal((M, K)) * 10.0 ** rng.integers(-4, 3, (M, K))).astype(np.float16)
    Qc = rng.integers(0, 16, size=(K, N), dtype=np.uint8)
    S = (10.0 ** rng.uniform(-6, 1.5, size=(K // G, N))).astype(np.float16)
    want = _exact_reference(A, Qc, S, G)
    got = oracle_lib.gemm(A, inputs.kpack(Qc), S, G)
    assert np.array_equal(got.view(np.uint16), want.view(np.uint16))


# ---------- P5: the library routine on the same definition ---------------------------------------

@pytest.mark.parametrize("M,K,N,G", [(1, 128, 128, 128), (7, 256, 192, 128), (16, 512, 256, 512), (33, 1024, 128, 128)])
def test_gemm_equals_numpy_fp64_matmul(oracle_lib, M, K, N, G):
    case = inputs.make_dense(M, K, N, G, 100 + M)
    Q = oracle_lib.unpack_q(case.q_kpacked).astype(np.int64)
    W = (Q - 8) * np.repeat(case.S.astype(np.float64), G, axis=0)  # integers times exact scales
    want = (case.A.astype(np.float64) @ W).astype(np.float16)
    got = oracle_lib.gemm(case.A, case.q_kpacked, case.S, G)
    assert np.array_equal(got.view(np.uint16), want.view(np.uint16))
    # and the one-output-at-a-time routine agrees with the full one
    rng = np.random.default_rng(5)
    ms = rng.integers(0, M, 200)
    ns = rng.integers(0, N, 200)
    samp = oracle_lib.gemm_samples(case.A, case.q_kpacked, case.S, G, ms, ns)
    assert np.array_equal(samp.view(np.uint16), got[ms, ns].view(np.uint16))


# ---------- P6 / P7: closed forms and one-hot probing ----------------------------------------------

def test_all_codes_eight_gives_zero(oracle_lib):
    case = inputs.make_dense(4, 256, 64, 128, 9)
    q8 = inputs.kpack(np.full((256, 64), 8, dtype=np.uint8))
    C = oracle_lib.gemm(case.A, q8, case.S, 128)
    assert np.all(C == 0)


def test_unit_activations_and_scales_give_integer_column_sums(oracle_lib):
    rng = np.random.default_rng(21)
    K, N = 4096, 32
    Q = rng.integers(0, 16, size=(K, N), dtype=np.uint8)
    A = np.ones((2, K), dtype=np.float16)
    S = np.ones((K // 128, N), dtype=np.float16)
    sums = (Q.astype(np.int64) - 8).sum(axis=0)  # integers, may exceed 2048 in magnitude
    want = np.array([_round_fraction_to_f16_bits(Fraction(int(v))) for v in sums], dtype=np.uint16)
    C = oracle_lib.gemm(A, inputs.kpack(Q), S, 128)
    assert np.array_equal(C[0].view(np.uint16), want)
    assert np.array_equal(C[1].view(np.uint16), want)


def test_one_hot_rows_read_back_single_weights(oracle_lib):
    # A = rows of the identity: C[m, n] = (Q[k_m, n] - 8) * S[k_m // G, n], scales distinct powers of two
    rng = np.random.default_rng(22)
    K, N, G = 256, 48, 64
    Q = rng.integers(0, 16, size=(K, N), dtype=np.uint8)
    expo = rng.integers(-6, 3, size=(K // G, N))
    S = np.ldexp(1.0, expo).astype(np.float16)
    ks = np.array([0, 1, 7, 8, 63, 64, 65, 127, 128, 200, 255])
    A = np.zeros((ks.size, K), dtype=np.float16)
    A[np.arange(ks.size), ks] = 1.0
    C = oracle_lib.gemm(A, inputs.kpack(Q), S, G)
    for i, k in enumerate(ks):
        want = (Q[k].astype(np.int64) - 8) * np.ldexp(1.0, expo[k // G])  # exact small numbers
        assert np.array_equal(C[i].astype(np.float64), want)


def test_negative_activation_flips_sign_and_operands_not_transposed(oracle_lib):
    # a non-square, asymmetric case with a hand-computable answer
    K, N = 16, 2
    Q = np.full((K, N), 8, dtype=np.uint8)
    Q[3, 0] = 15   # +7
    Q[5, 1] = 0    # -8
    A = np.zeros((3, K), dtype=np.float16)
    A[0, 3] = 2.0
    A[1, 5] = -0.5
    A[2, 3] = 1.0
    A[2, 5] = 1.0
    S = np.array([[0.5, 0.25]], dtype=np.float16)
    C = oracle_lib.gemm(A, inputs.kpack(Q), S, 16).astype(np.float64)
    assert np.array_equal(C, np.array([[7.0, 0.0], [0.0, 1.0], [3.5, -2.0]]))


# ---------- P9: the 2:4 form ----------------------------------------------------------------------

def _expand_numpy(case):
    K, N = case.K, case.N
    Qc = np.zeros((K // 2, N), dtype=np.uint8)
    for j in range(8):
        Qc[j::8, :] = (case.qc_kpacked >> np.uint32(4 * j)) & 15
    Q = np.full((K, N), 8, dtype=np.uint8)
    t = np.arange(K // 2)
    rows = 4 * (t // 2)[:, None] + case.idx
    Q[rows, np.arange(N)[None, :]] = Qc
    return Q


@pytest.mark.parametrize("M,K,N,G", [(2, 64, 16, 32), (5, 256, 128, 128), (3, 128, 40, 128)])
def test_sparse24_equals_dense_with_zeros(oracle_lib, M, K, N, G):
    case = inputs.make_sparse24(M, K, N, G, 40 + M)
    Q = _expand_numpy(case)
    # exactly two kept positions per group of four, everything else is the zero code
    assert np.array_equal(oracle_lib.sparse24_expand(case.qc_kpacked, case.idx), Q)
    dense = oracle_lib.gemm(case.A, inputs.kpack(Q), case.S, G)
    sparse = oracle_lib.gemm_sparse24(case.A, case.qc_kpacked, case.idx, case.S, G)
    assert np.array_equal(dense.view(np.uint16), sparse.view(np.uint16))


def test_sparse24_tiny_exact(oracle_lib):
    case = inputs.make_sparse24(2, 32, 3, 16, 77)
    want = _exact_reference(case.A, _expand_numpy(case), case.S, 16)
    got = oracle_lib.gemm_sparse24(case.A, case.qc_kpacked, case.idx, case.S, 16)
    assert np.array_equal(got.view(np.uint16), want.view(np.uint16))


def test_sparse24_rejects_unordered_indices(oracle_lib):
    case = inputs.make_sparse24(1, 32, 2, 32, 1)
    bad = case.idx.copy()
    bad[0, 0], bad[1, 0] = 3, 1
    with pytest.raises(RuntimeError):
        oracle_lib.sparse24_expand(case.qc_kpacked, bad)


# ---------- the acceptance bound itself -----------------------------------------------------------

def test_tolerance_checker(oracle_lib):
    ref = np.array([[1.0, -2.0, 0.0, 4.0]], dtype=np.float16)
    rms = np.sqrt((1 + 4 + 0 + 16) / 4)
    bad, worst, got_rms = oracle_lib.check_tolerance(ref.copy(), ref)
    assert bad == 0 and worst == 0 and abs(got_rms - rms) < 1e-12
    c = ref.copy()
    c[0, 2] = np.float16(0.011)  # allowance at 0 is 5e-3 * rms = 0.01146
    assert oracle_lib.check_tolerance(c, ref)[0] == 0
    c[0, 2] = np.float16(0.012)
    assert oracle_lib.check_tolerance(c, ref)[0] == 1
    c = ref.copy()
    c[0, 3] = np.float16(np.inf)
    assert oracle_lib.check_tolerance(c, ref)[0] == 1
    c[0, 3] = np.float16(np.nan)
    assert oracle_lib.check_tolerance(c, ref)[0] == 1


def test_generator_recipe_and_seeds():
    a = inputs.make_dense(16, 256, 128, 128, 0)
    b = inputs.make_dense(16, 256, 128, 128, 0)
    assert np.array_equal(a.A, b.A) and np.array_equal(a.q_kpacked, b.q_kpacked) and np.array_equal(a.S, b.S)
    assert a.S.min() >= np.float16(0.005) and a.S.max() <= np.float16(0.02)
    assert abs(float(a.A.astype(np.float64).std()) - 1.0) < 0.05
    s = inputs.make_sparse24(1, 256, 64, 128, 5)
    assert np.all(s.idx[0::2] < s.idx[1::2]) and s.idx.max() <= 3
    cases = list(inputs.iter_cases(4))
    assert len(cases) == 3 * 2 * 4 and len({c[-1] for c in cases}) == len(cases)
    assert list(inputs.iter_cases(1)) == [("single", 16, 4096, 4096, 128, 0)]


def test_sparse24_literal_case_typed_out_by_hand(oracle_lib):
    # Section 2.2 / Section 4: in every group of four consecutive rows of a column two values are kept, each with
    # its 2-bit position inside the group; everything else is zero.  K = 16, N = 2, scale groups of 8 rows.
    # Every number below was written out by hand from that definition (no formula of the oracle is re-used).
    #
    # kept values (code, position) in the order they are stored, four groups per column:
    #   column 0: (15,1) (0,3) | (9,0) (6,2) | (8,0) (11,3) | (7,1) (8,2)
    #   column 1: (8,0) (12,1) | (3,2) (10,3) | (15,1) (1,2) | (0,0) (9,3)
    qc = np.array([[0x87B8690F, 0x901FA3C8]], dtype=np.uint32)   # nibble t of a word = code of kept value t
    idx = np.array([[1, 0], [3, 1], [0, 2], [2, 3], [0, 1], [3, 2], [1, 0], [2, 3]], dtype=np.uint8)
    # the dense codes this stands for (8 = the zero code at pruned positions)
    Q = np.array([[8, 8], [15, 12], [8, 8], [0, 8],
                  [9, 8], [8, 8], [6, 3], [8, 10],
                  [8, 8], [8, 15], [8, 1], [11, 8],
                  [8, 0], [7, 8], [8, 8], [8, 9]], dtype=np.uint8)
    assert np.array_equal(oracle_lib.sparse24_expand(qc, idx), Q)
    S = np.array([[0.5, 0.25], [2.0, 1.0]], dtype=np.float16)
    A = np.array([[1, 2, 3, 4, 5, 6, 7, 8, 1, 1, 1, 1, 2, 2, 2, 2],
                  [-1, 0, 0, 0.5, 0, 0, 0, -2, 0, 0, 3, 0, 0, -1, 0, 0.25]], dtype=np.float16)
    # row 0, column 0: 0.5 * (2*7 + 4*(-8) + 5*1 + 7*(-2)) + 2 * (1*3 + 2*(-1)) = -13.5 + 2 = -11.5
    # row 0, column 1: 0.25 * (2*4 + 7*(-5) + 8*2) + 1 * (7 - 7 + 2*(-8) + 2*1) = -2.75 - 14 = -16.75
    # row 1, column 0: 0.5 * (0.5*(-8)) + 2 * ((-1)*(-1)) = -2 + 2 = 0
    # row 1, column 1: 0.25 * ((-2)*2) + 1 * (3*(-7) + 0.25*1) = -1 - 20.75 = -21.75
    want = np.array([[-11.5, -16.75], [0.0, -21.75]])
    got = oracle_lib.gemm_sparse24(A, qc, idx, S, 8).astype(np.float64)
    assert np.array_equal(got, want)
