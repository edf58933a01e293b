"""Pins for the oracle's linear layer (Eq. 3: h = Linear(concat[e, f]); the decoder layer's projections), RMS
normalisation and embedding lookup.  Expected values come from plain Python loops on integer inputs and from identities a
correct implementation must satisfy; none re-calls the oracle's own matrix product."""
import math

import numpy as np
import pytest

import oracle


def test_concat_linear_by_plain_loops():
    rng = np.random.default_rng(1)
    R, K1, K2, N = 3, 4, 5, 6
    e, f = rng.integers(-3, 4, (R, K1)), rng.integers(-3, 4, (R, K2))
    w, b = rng.integers(-3, 4, (N, K1 + K2)), rng.integers(-3, 4, N)
    got = oracle.linear(e, w, x2=f, bias=b)
    for r in range(R):
        for n in range(N):
            want = int(b[n]) + sum(int(e[r, k]) * int(w[n, k]) for k in range(K1)) + sum(int(f[r, k]) * int(w[n, K1 + k]) for k in range(K2))
            assert got[r, n] == want            # exact: small integers; the second input meets the LAST K2 columns of w


def test_gate_and_residual_by_plain_loops():
    rng = np.random.default_rng(2)
    R, K, N = 4, 5, 3
    x, w, res = rng.integers(-2, 3, (R, K)), rng.integers(-2, 3, (2 * N, K)), rng.integers(-5, 6, (R, N))
    got = oracle.linear(x, w, residual=res, gate=True)
    for r in range(R):
        for n in range(N):
            g = sum(int(x[r, k]) * int(w[n, k]) for k in range(K))            # gate rows first ...
            u = sum(int(x[r, k]) * int(w[N + n, k]) for k in range(K))        # ... then the up rows
            want = g / (1.0 + math.exp(-g)) * u + int(res[r, n])
            assert got[r, n] == pytest.approx(want, abs=1e-12)
    assert oracle.linear(np.zeros((1, K)), w, gate=True).tolist() == [[0.0] * N]   # silu(0) * 0


def test_rmsnorm_properties():
    rng = np.random.default_rng(3)
    x, g = rng.standard_normal((6, 32)), rng.standard_normal(32)
    y = oracle.rmsnorm(x, np.ones(32), eps=0.0)
    np.testing.assert_allclose(np.mean(y * y, axis=1), 1.0, rtol=1e-13)                       # unit mean square
    np.testing.assert_allclose(oracle.rmsnorm(7.5 * x, g, eps=0.0), oracle.rmsnorm(x, g, eps=0.0), rtol=1e-13)   # scale-free
    np.testing.assert_allclose(oracle.rmsnorm(x, g, eps=0.0), y * g, rtol=1e-13)             # the weight multiplies
    one = oracle.rmsnorm(np.array([[3.0, 4.0]]), np.array([1.0, 1.0]), eps=0.0)               # rms = sqrt(12.5)
    np.testing.assert_allclose(one, [[3.0 / math.sqrt(12.5), 4.0 / math.sqrt(12.5)]], rtol=1e-15)
    assert np.all(np.abs(oracle.rmsnorm(np.zeros((1, 4)), np.ones(4), eps=1e-6)) == 0.0)      # eps keeps 0 / 0 away


def test_embedding_rows():
    table = np.arange(20).reshape(5, 4)
    np.testing.assert_array_equal(oracle.embed_gather(table, [4, 0, 4]), [[16, 17, 18, 19], [0, 1, 2, 3], [16, 17, 18, 19]])
