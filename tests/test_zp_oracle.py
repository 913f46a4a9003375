"""Pins of the zero-point oracle (oracle/zp_ref.py): the symmetric special case, a hand-worked literal, exact rational
arithmetic on a small case, linearity in the zero points.  No GPU."""
from fractions import Fraction

import numpy as np

import oracle
from oracle import zp_ref
from paper_2408_11743_b200 import inputs


def test_zero_point_eight_is_the_symmetric_layer():
    # integer-valued inputs: every sum is exact in fp64 in any order, so the two oracles must agree bit for bit
    rng = np.random.default_rng(0)
    K, N, G, M = 256, 64, 128, 5
    Q = rng.integers(0, 16, size=(K, N), dtype=np.uint8)
    A = rng.integers(-4, 5, size=(M, K)).astype(np.float16)
    S = np.ldexp(1.0, rng.integers(-5, 2, size=(K // G, N))).astype(np.float16)
    q = inputs.kpack(Q)
    Z = np.full((K // G, N), 8, dtype=np.uint8)
    assert np.array_equal(zp_ref.gemm_zp(A, q, S, Z, G).view(np.uint16), oracle.gemm(A, q, S, G).view(np.uint16))


def test_hand_worked_literal():
    # one row of A, two groups of 8 rows, two columns; worked by hand:
    #   column 0: group 0 codes 0..7 with z = 3, s = 0.5: (q - 3) = -3..4, A = 1 everywhere -> 0.5 * 4 = 2
    #             group 1 codes all 15 with z = 15, s = 2: zero contribution
    #   column 1: group 0 codes all 0 with z = 0: zero; group 1 codes 8..15 with z = 8, s = 0.25, A = 2 -> 2 * 0.25 * 28 = 14
    Q = np.zeros((16, 2), dtype=np.uint8)
    Q[:8, 0] = np.arange(8)
    Q[8:, 0] = 15
    Q[8:, 1] = np.arange(8, 16)
    Z = np.array([[3, 0], [15, 8]], dtype=np.uint8)
    S = np.array([[0.5, 1.0], [2.0, 0.25]], dtype=np.float16)
    A = np.ones((1, 16), dtype=np.float16)
    A[0, 8:] = 2
    W = zp_ref.dequant_zp(Q, S, Z, 8)
    C = A.astype(np.float64) @ W
    assert C.tolist() == [[2.0, 14.0]]
    assert W[0, 0] == -1.5 and W[7, 0] == 2.0 and W[15, 1] == 1.75


def test_exact_rational_arithmetic_on_a_small_case():
    rng = np.random.default_rng(2)
    K, N, G, M = 64, 8, 32, 3
    Q = rng.integers(0, 16, size=(K, N), dtype=np.uint8)
    Z = rng.integers(0, 16, size=(K // G, N), dtype=np.uint8)
    S = rng.uniform(0.01, 0.1, size=(K // G, N)).astype(np.float16)
    A = rng.standard_normal((M, K)).astype(np.float16)
    C = zp_ref.gemm_zp(A, inputs.kpack(Q), S, Z, G)
    for m in range(M):
        for n in range(N):
            acc = Fraction(0)
            for k in range(K):
                acc += Fraction(float(A[m, k])) * (int(Q[k, n]) - int(Z[k // G, n])) * Fraction(float(S[k // G, n]))
            # the fp16 nearest to the exact sum (ties cannot be told apart from float(acc) alone, so allow one ulp there)
            want = np.float16(float(acc))
            assert abs(float(C[m, n]) - float(want)) <= float(np.spacing(want)) * (float(C[m, n]) != float(want))
            assert abs(float(C[m, n]) - float(acc)) <= 0.5 * float(np.spacing(np.float16(abs(float(acc))))) * (1 + 1e-9)


def test_linear_in_the_zero_points():
    # C(Z) - C(Z') = A . ((Z' - Z) * S) group by group: with integer-valued A and power-of-two scales all of it is exact
    rng = np.random.default_rng(3)
    K, N, G, M = 128, 16, 32, 4
    Q = rng.integers(0, 16, size=(K, N), dtype=np.uint8)
    A = rng.integers(-2, 3, size=(M, K)).astype(np.float16)
    S = np.ldexp(1.0, rng.integers(-3, 1, size=(K // G, N))).astype(np.float16)
    Z1 = rng.integers(0, 16, size=(K // G, N), dtype=np.uint8)
    Z2 = rng.integers(0, 16, size=(K // G, N), dtype=np.uint8)
    q = inputs.kpack(Q)
    C1 = zp_ref.gemm_zp(A, q, S, Z1, G).astype(np.float64)
    C2 = zp_ref.gemm_zp(A, q, S, Z2, G).astype(np.float64)
    asum = A.astype(np.float64).reshape(M, K // G, G).sum(axis=2)  # [M, groups]
    diff = asum @ ((Z2.astype(np.float64) - Z1.astype(np.float64)) * S.astype(np.float64))
    assert np.array_equal(C1 - C2, diff)
