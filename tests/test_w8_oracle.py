"""Pins of the 8-bit oracle (oracle/w8_ref.py).  No GPU."""
from fractions import Fraction

import numpy as np

import oracle
from oracle import w8_ref
from paper_2408_11743_b200 import inputs


def test_codes_that_fit_four_bits_reproduce_the_four_bit_layer():
    # q8 = 120 + q4 gives q8 - 128 = q4 - 8: the two oracles must agree bit for bit on integer-valued inputs
    rng = np.random.default_rng(0)
    K, N, G, M = 256, 64, 128, 5
    Q4 = rng.integers(0, 16, size=(K, N), dtype=np.uint8)
    A = rng.integers(-4, 5, size=(M, K)).astype(np.float16)
    S = np.ldexp(1.0, rng.integers(-5, 2, size=(K // G, N))).astype(np.float16)
    C8 = w8_ref.gemm_w8(A, (Q4 + 120).astype(np.uint8), S, G)
    assert np.array_equal(C8.view(np.uint16), oracle.gemm(A, inputs.kpack(Q4), S, G).view(np.uint16))


def test_hand_worked_literal():
    # K = 4, one group, two columns: column 0 codes (0, 128, 255, 129) -> (-128, 0, 127, 1) * 0.5; A = (1, 5, 2, -4)
    #   -> 0.5 * (-128 + 0 + 254 - 4) = 61; column 1 codes all 128 -> 0
    Q8 = np.array([[0, 128], [128, 128], [255, 128], [129, 128]], dtype=np.uint8)
    S = np.array([[0.5, 3.0]], dtype=np.float16)
    A = np.array([[1, 5, 2, -4]], dtype=np.float16)
    W = w8_ref.dequant_w8(Q8, S, 4)
    assert W[:, 0].tolist() == [-64.0, 0.0, 63.5, 0.5]
    assert (A.astype(np.float64) @ W).tolist() == [[61.0, 0.0]]


def test_exact_rational_arithmetic_on_a_small_case():
    rng = np.random.default_rng(2)
    K, N, G, M = 64, 6, 32, 3
    Q8 = rng.integers(0, 256, size=(K, N), dtype=np.uint8)
    S = rng.uniform(0.001, 0.01, size=(K // G, N)).astype(np.float16)
    A = rng.standard_normal((M, K)).astype(np.float16)
    C = w8_ref.gemm_w8(A, Q8, S, G)
    for m in range(M):
        for n in range(N):
            acc = sum(Fraction(float(A[m, k])) * (int(Q8[k, n]) - 128) * Fraction(float(S[k // G, n])) for k in range(K))
            assert abs(float(C[m, n]) - float(acc)) <= 0.5 * float(np.spacing(np.float16(abs(float(acc))))) * (1 + 1e-9)


def test_packed_order_places_marked_codes_where_the_description_says():
    K, N = 256, 512
    Q8 = np.zeros((K, N), dtype=np.uint8)
    marks = [(0, 0, 1), (17, 3, 2), (130, 300, 3), (255, 511, 4), (128 + 16 * 5 + 7, 256 + 9, 5)]
    for k, n, v in marks:
        Q8[k, n] = v
    P = w8_ref.pack_w8(Q8)
    for k, n, v in marks:
        T, nn, kb, c, j = n // 256, n % 256, k // 128, (k % 128) // 16, k % 16
        assert P[(((T * (K // 128) + kb) * 8 + c) * 256 + nn) * 16 + j] == v
    assert np.count_nonzero(P) == len(marks)
