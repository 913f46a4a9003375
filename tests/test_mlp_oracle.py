"""Pins of the MLP-chain oracle (oracle/mlp_ref.py).  No GPU."""
import math

import numpy as np

from oracle import mlp_ref


def test_silu_values_and_identities():
    assert mlp_ref.silu(np.array([0.0]))[0] == 0.0
    assert abs(mlp_ref.silu(np.array([1.0]))[0] - 1.0 / (1.0 + math.exp(-1.0))) < 1e-15
    assert abs(mlp_ref.silu(np.array([-2.0]))[0] + 2.0 / (1.0 + math.exp(2.0))) < 1e-15
    x = np.linspace(-12, 12, 1001)
    assert np.allclose(mlp_ref.silu(x) - mlp_ref.silu(-x), x, atol=1e-13)       # silu(x) - silu(-x) = x
    assert np.allclose(mlp_ref.silu(np.array([40.0, -40.0])), [40.0, 0.0], atol=1e-15)
    assert mlp_ref.silu(x).min() > -0.2785 and abs(mlp_ref.silu(x).min() + 0.27846) < 1e-4  # the minimum of silu


def test_swiglu_literal_and_rounding():
    g = np.array([[0.0, 1.0, -1.0, 8.0]], dtype=np.float16)
    u = np.array([[3.0, 2.0, 2.0, 0.5]], dtype=np.float16)
    h = mlp_ref.swiglu(g, u).astype(np.float64)[0]
    want = [0.0, 2.0 * 0.7310585786300049, -2.0 * 0.2689414213699951, 4.0 * 0.9996646498695336]
    for a, b in zip(h, want):
        assert abs(a - b) <= 0.5 * float(np.spacing(np.float16(abs(b)))) + 1e-12


def test_interleave_is_blocks_of_eight_gate_then_eight_up():
    I = 32
    gate = np.arange(I, dtype=np.int32)[None, :]            # gate channel c -> c
    up = 1000 + np.arange(I, dtype=np.int32)[None, :]       # up channel c -> 1000 + c
    out = mlp_ref.interleave(gate, up)[0]
    for n in range(2 * I):
        b, r = divmod(n, 16)
        assert out[n] == (8 * b + r if r < 8 else 1000 + 8 * b + r - 8)
