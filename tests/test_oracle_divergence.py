"""Pins for the oracle's aggregation divergence (Section 4.3, Definition 2, Eq. 7)."""
from fractions import Fraction
import math

import numpy as np
import pytest

import oracle


def brute(models, weights, mean_of=None):
    """rho_i^2 in exact rationals, written per worker with plain Python sums."""
    src = models if mean_of is None else mean_of
    N, P = models.shape
    D = [Fraction(float(w)) for w in weights] if weights is not None else [Fraction(1)] * N
    tot = sum(D)
    out = []
    for i in range(N):
        acc = Fraction(0)
        for p in range(P):
            mean = sum(D[j] * Fraction(float(src[j, p])) for j in range(N)) / tot
            acc += (Fraction(float(models[i, p])) - mean) ** 2
        out.append(math.sqrt(acc))
    return np.array(out)


@pytest.mark.parametrize("N,P", [(1, 5), (2, 7), (3, 16), (5, 33)])
def test_brute_force(N, P):
    rng = np.random.default_rng(N + P)
    x = rng.normal(0, 0.05, (N, P)).astype(np.float32)
    y = rng.normal(0, 0.05, (N, P)).astype(np.float32)
    w = rng.integers(500, 1501, N).astype(np.float32)
    for weights in (None, w):
        np.testing.assert_allclose(oracle.divergence(x, weights), brute(x, weights), rtol=1e-13, atol=1e-18)
        np.testing.assert_allclose(oracle.divergence(x, weights, mean_of=y), brute(x, weights, y), rtol=1e-13)


def test_two_workers_closed_form():
    # mean = (D1 x + D2 y)/(D1+D2)  =>  rho_1 = D2/(D1+D2) ||x-y||, rho_2 = D1/(D1+D2) ||x-y||
    rng = np.random.default_rng(0)
    x = rng.normal(0, 1, (2, 40)).astype(np.float32)
    dist = np.linalg.norm(x[0].astype(np.float64) - x[1].astype(np.float64))
    rho = oracle.divergence(x, np.array([1.0, 3.0], dtype=np.float32))
    np.testing.assert_allclose(rho, [0.75 * dist, 0.25 * dist], rtol=1e-14)
    rho = oracle.divergence(x)
    np.testing.assert_allclose(rho, [0.5 * dist, 0.5 * dist], rtol=1e-14)


def test_hand_example():
    # three workers, two parameters, equal weights: mean = (2, 1)
    x = np.array([[0, 1], [2, 4], [4, -2]], dtype=np.float32)
    np.testing.assert_allclose(oracle.divergence(x), [2.0, 3.0, math.sqrt(13.0)], rtol=1e-15)
    # weights 1,1,2: mean = (2.5, 0.25)
    rho = oracle.divergence(x, np.array([1, 1, 2], dtype=np.float32))
    np.testing.assert_allclose(rho, [math.hypot(2.5, 0.75), math.hypot(0.5, 3.75), math.hypot(1.5, 2.25)], rtol=1e-15)


def test_identical_models_have_zero_divergence():
    row = np.random.default_rng(1).normal(0, 0.05, (1, 50)).astype(np.float32)
    x = np.repeat(row, 6, axis=0)
    assert (oracle.divergence(x, np.arange(1, 7, dtype=np.float32)) <= 1e-9).all()


def test_translation_and_scaling_laws():
    rng = np.random.default_rng(2)
    x = rng.integers(-8, 9, (4, 30)).astype(np.float32)          # small integers: exact arithmetic
    w = np.array([1, 2, 3, 2], dtype=np.float32)
    base = oracle.divergence(x, w)
    np.testing.assert_allclose(oracle.divergence(x + 16.0, w), base, rtol=1e-14)   # shift invariant
    np.testing.assert_allclose(oracle.divergence(x * 4.0, w), 4.0 * base, rtol=1e-14)
    np.testing.assert_allclose(oracle.divergence(x, w * 8.0), base, rtol=1e-14)    # weights are relative


def test_full_replica_round_has_zero_divergence_and_more_replicas_shrink_it():
    # Section 4.3: with R = n-1 no divergence is left, and pulling more replicas per segment
    # shrinks it
    rng = np.random.default_rng(3)
    N, P, S = 10, 400, 5
    x = rng.normal(0, 0.05, (N, P)).astype(np.float32)
    w = rng.integers(500, 1501, N).astype(np.float32)
    scale = np.linalg.norm(x[0])
    means = []
    for R in (1, 2, 4, N - 1):
        rho = np.zeros(N)
        for seed in range(8):
            idx = oracle.select_peers(seed, 0, N, S, R)
            out = oracle.segment_aggregate(x, idx, S, R, weights=w).astype(np.float32)
            rho += oracle.divergence(out, w, mean_of=x)
        means.append(rho.mean() / 8)
    assert means[0] > means[1] > means[2] > means[3]
    assert means[3] <= 1e-6 * scale
