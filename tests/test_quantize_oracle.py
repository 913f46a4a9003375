"""Pins of the quantiser oracle (oracle/quantize_oracle.c): hand-worked literal cases, exact rational brute force on
small groups, bounds that follow from the definition, invariances.  No GPU."""
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import quantize_ref

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "quantize_literal.txt")


def _cases():
    rows = [l.strip() for l in open(GOLDEN) if l.strip() and not l.startswith("#")]
    out = []
    for i in range(0, len(rows), 6):
        name = rows[i]
        n_grid, n_cand = (int(x) for x in rows[i + 1].split())
        w = [float(x) for x in rows[i + 2].split()]
        codes = [int(x) for x in rows[i + 3].split()]
        out.append((name, n_grid, n_cand, w, codes, float(rows[i + 4]), int(rows[i + 5])))
    return out


@pytest.mark.parametrize("case", _cases(), ids=lambda c: c[0])
def test_hand_worked_cases(case):
    name, n_grid, n_cand, w, codes, scale, chosen = case
    s0 = 2.0 ** -6
    W = (np.array(w, dtype=np.float64) * s0).astype(np.float16).reshape(-1, 1)
    assert np.array_equal(W.astype(np.float64).ravel(), np.array(w) * s0)  # the case is exactly representable
    Q, S, T = quantize_ref.quantize_rtn(W, len(w), n_grid, n_cand)
    assert Q.ravel().tolist() == codes
    assert float(S[0, 0]) == scale * s0
    assert int(T[0, 0]) == chosen


def _f16_frac(h):
    return Fraction(float(h))


def _exact_candidate(w, s):
    """codes and exact squared error of one candidate scale, in rational arithmetic (round half to even)."""
    err = Fraction(0)
    codes = []
    for x in w:
        t = x / s
        fl = t.numerator // t.denominator
        rem = t - fl
        q = fl + (1 if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and fl % 2 == 1) else 0)
        q = max(-8, min(7, q))
        codes.append(q + 8)
        err += (x - q * s) ** 2
    return codes, err


def test_brute_force_in_rational_arithmetic_on_small_groups():
    # the winner must be the candidate with the least EXACT error whenever the exact errors are well apart, and the
    # codes must be the exactly rounded ones except where w / s falls within fp32 rounding of a half-way point
    rng = np.random.default_rng(0)
    G, N, n_grid, n_cand = 16, 40, 10, 6
    W = (rng.standard_normal((G, N)) * 0.05).astype(np.float16)
    W[3, ::5] *= 6  # some outliers
    Q, S, T = quantize_ref.quantize_rtn(W, G, n_grid, n_cand)
    for n in range(N):
        w = [_f16_frac(x) for x in W[:, n]]
        a = max(abs(x) for x in w)
        errs, code_sets, scales = [], [], []
        for t in range(n_cand):
            s_exact = 2 * a * (1 - Fraction(t, n_grid)) / 15
            s16 = np.float16(float(s_exact))  # correctly rounded: float(Fraction) is exact to fp64, far finer than fp16
            scales.append(s16)
            c, e = _exact_candidate(w, _f16_frac(s16))
            code_sets.append(c)
            errs.append(e)
        best = min(range(n_cand), key=lambda t: (errs[t], t))
        order = sorted(errs)
        if len(order) > 1 and order[1] > order[0] * (1 + Fraction(1, 10**4)):
            assert int(T[0, n]) == best, (n, [float(e) for e in errs])
        t = int(T[0, n])
        # the scale may differ from the exactly rounded one by one fp16 step at most (it is computed in fp32)
        assert abs(float(S[0, n]) - float(scales[t])) <= float(np.spacing(scales[t]))
        if float(S[0, n]) == float(scales[t]):
            ties = sum(1 for x in w if ((x / _f16_frac(scales[t])) * 2).denominator == 1)
            mism = sum(int(a_ != b_) for a_, b_ in zip(Q[:, n].tolist(), code_sets[t]))
            assert mism <= ties


@pytest.mark.parametrize("G,n_grid,n_cand", [(32, 20, 10), (128, 20, 10), (128, 8, 8), (256, 20, 1), (64, 5, 3)])
def test_bounds_that_follow_from_the_definition(G, n_grid, n_cand):
    rng = np.random.default_rng(G + n_cand)
    K, N = 4 * G, 48
    W = (rng.standard_normal((K, N)) * 0.02).astype(np.float16)
    W[rng.integers(0, K, 40), rng.integers(0, N, 40)] *= 8  # outliers
    Q, S, T = quantize_ref.quantize_rtn(W, G, n_grid, n_cand)
    assert Q.min() >= 0 and Q.max() <= 15 and np.all(S.astype(np.float64) > 0)
    assert T.min() >= 0 and T.max() < n_cand
    Wd = W.astype(np.float64)
    Sd = np.repeat(S.astype(np.float64), G, axis=0)
    deq = (Q.astype(np.float64) - 8) * Sd
    inside = (Wd >= -8.5 * Sd) & (Wd <= 7.5 * Sd)
    # round to nearest: half a step inside the grid's range; outside it the code is the end of the grid
    assert np.all(np.abs(Wd - deq)[inside] <= 0.5 * Sd[inside] * (1 + 1e-6))
    assert np.all(Q[Wd > 7.5 * Sd] == 15) and np.all(Q[Wd < -8.5 * Sd] == 0)
    # the scale is 2 a r / 15 for the chosen candidate, to fp16 precision
    a = np.abs(Wd).reshape(K // G, G, N).max(axis=1)
    want = 2 * a * (1 - T / n_grid) / 15
    assert np.allclose(S.astype(np.float64), want, rtol=2.0 ** -10, atol=2.0 ** -24)
    # the chosen candidate has the least error among all of them, evaluated independently in fp64 with numpy
    Wg = Wd.reshape(K // G, G, N)
    best = None
    for t in range(n_cand):
        s = (2 * a.astype(np.float32) * np.float32(1 - t / n_grid) / 15).astype(np.float16).astype(np.float64)
        s = np.maximum(s, 2.0 ** -24)
        q = np.clip(np.rint(Wg / s[:, None, :]), -8, 7)
        e = ((Wg - q * s[:, None, :]) ** 2).sum(axis=1)
        best = e if best is None else np.minimum(best, e)
    got = ((Wd - deq) ** 2).reshape(K // G, G, N).sum(axis=1)
    assert np.all(got <= best * (1 + 1e-4) + 1e-12)
    if n_cand == 1:
        assert np.all(T == 0)


def test_scaling_by_powers_of_two_changes_only_the_scales():
    rng = np.random.default_rng(5)
    W = (rng.standard_normal((256, 32)) * 0.03).astype(np.float16)
    Q, S, T = quantize_ref.quantize_rtn(W, 128, 20, 10)
    for k in (-3, 2, 5):
        W2 = (W.astype(np.float32) * 2.0 ** k).astype(np.float16)
        Q2, S2, T2 = quantize_ref.quantize_rtn(W2, 128, 20, 10)
        assert np.array_equal(Q, Q2) and np.array_equal(T, T2)
        assert np.array_equal(S2.astype(np.float64), S.astype(np.float64) * 2.0 ** k)


def test_search_never_loses_to_plain_rounding_and_wins_on_outliers():
    rng = np.random.default_rng(6)
    W = (rng.standard_normal((512, 64)) * 0.02).astype(np.float16)
    W[::128, :] *= 3  # one moderate outlier per group: clipping it lets the other 127 weights use a finer grid
    Wd = W.astype(np.float64)

    def sq_err(n_cand):
        Q, S, _ = quantize_ref.quantize_rtn(W, 128, 20, n_cand)
        return ((Wd - (Q.astype(np.float64) - 8) * np.repeat(S.astype(np.float64), 128, axis=0)) ** 2).reshape(4, 128, 64).sum(axis=1)
    plain, searched = sq_err(1), sq_err(10)
    assert np.all(searched <= plain * (1 + 1e-5))
    assert searched.sum() < 0.9 * plain.sum()


def test_bad_arguments_are_refused():
    W = np.zeros((128, 8), dtype=np.float16)
    for args in [(100, 20, 10), (128, 0, 1), (128, 4, 5), (128, 4, 0)]:
        with pytest.raises(ValueError):
            quantize_ref.quantize_rtn(W, *args)
    with pytest.raises(ValueError):
        quantize_ref.quantize_rtn(np.full((128, 8), np.inf, dtype=np.float16), 128)
