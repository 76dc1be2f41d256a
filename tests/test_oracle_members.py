"""Pins for the oracle's dynamic-worker variants (Section 4.2): offline workers are not
pulled from, newcomers aggregate without their local model."""
from fractions import Fraction

import numpy as np
import pytest

import oracle


@pytest.mark.parametrize("N,S,R", [(8, 4, 2), (5, 9, 4), (33, 2, 7), (4, 5, 3), (2, 3, 1)])
def test_all_online_equals_plain_sampler(N, S, R):
    for seed, rnd in ((1, 0), (9, 4)):
        a = oracle.select_peers(seed, rnd, N, S, R)
        assert (oracle.select_peers_active(seed, rnd, N, S, R) == a).all()
        assert (oracle.select_peers_active(seed, rnd, N, S, R, np.ones(N, np.uint8)) == a).all()


@pytest.mark.parametrize("N,S,R", [(8, 4, 2), (12, 5, 3), (33, 3, 6), (6, 7, 2)])
def test_offline_workers_are_never_pulled_from(N, S, R):
    rng = np.random.default_rng(N + S)
    for trial in range(6):
        active = np.ones(N, np.uint8)
        off = rng.choice(N, size=min(N - R - 1, 1 + trial % 3), replace=False)
        active[off] = 0
        idx = oracle.select_peers_active(trial, 2, N, S, R, active)
        n_on = int(active.sum())
        for w in range(N):
            if not active[w]:
                assert (idx[w] == -1).all()                 # an offline worker issues no request
                continue
            flat = idx[w].ravel()
            assert (flat >= 0).all() and (flat < N).all()
            assert active[flat].all() and not (flat == w).any()
            for l in range(S):
                assert (np.diff(idx[w, l]) > 0).all()
            use = np.bincount(flat, minlength=N)[active.astype(bool)]
            use = np.delete(use, np.flatnonzero(np.flatnonzero(active) == w))
            assert use.max() - use.min() <= 1                # spread evenly over the online others
            if S * R <= n_on - 2 + 1:
                assert len(set(flat.tolist())) == S * R


def test_masked_sampler_errors_and_uniformity():
    with pytest.raises(ValueError):
        oracle.select_peers_active(1, 0, 4, 2, 3, np.array([1, 1, 1, 0], np.uint8))   # only 2 online others
    # first draw uniform over the online others
    active = np.array([1, 0, 1, 1, 0, 1, 1], np.uint8)
    hist = np.zeros(7)
    for seed in range(4000):
        hist[oracle.select_peers_active(seed, 0, 7, 1, 1, active)[0, 0, 0]] += 1
    assert hist[[0, 1, 4]].sum() == 0
    exp = 1000.0
    assert (((hist[[2, 3, 5, 6]] - exp) ** 2) / exp).sum() < 22.0      # 3 dof


def brute(x, idx, S, R, weights, newcomer):
    N, P = x.shape
    L = -(-P // S)
    out = np.zeros((N, P))
    for w in range(N):
        for p in range(P):
            l = p // L
            prov = set() if (newcomer is not None and newcomer[w]) else {w}
            prov |= {int(k) for k in idx[w, l] if k >= 0}
            if not prov:
                prov = {w}
            num = sum(Fraction(float(weights[j])) * Fraction(float(x[j, p])) for j in prov)
            den = sum(Fraction(float(weights[j])) for j in prov)
            out[w, p] = float(num / den)
    return out


def test_members_reduce_to_plain_aggregation():
    rng = np.random.default_rng(0)
    N, P, S, R = 6, 41, 4, 2
    x = rng.normal(0, 0.05, (N, P)).astype(np.float32)
    w = rng.integers(500, 1501, N).astype(np.float32)
    idx = oracle.select_peers(1, 0, N, S, R)
    assert (oracle.segment_aggregate_members(x, idx, S, R, w) == oracle.segment_aggregate(x, idx, S, R, weights=w)).all()
    a = oracle.segment_aggregate_members(x, idx, S, R, w, ordered=True)
    b = oracle.segment_aggregate_ordered_f32(x, idx, S, R, weights=w)
    assert (a.view(np.uint32) == b.view(np.uint32)).all()


@pytest.mark.parametrize("seed", range(5))
def test_members_brute_force(seed):
    rng = np.random.default_rng(seed)
    N, P, S, R = 7, 30, 3, 3
    x = rng.normal(0, 0.05, (N, P)).astype(np.float32)
    w = rng.integers(500, 1501, N).astype(np.float32)
    active = np.ones(N, np.uint8)
    active[rng.choice(N, 2, replace=False)] = 0
    newcomer = np.zeros(N, np.uint8)
    newcomer[rng.choice(np.flatnonzero(active), 2, replace=False)] = 1
    idx = oracle.select_peers_active(seed, 1, N, S, R, active)
    idx[int(np.flatnonzero(active)[0]), 1, 0] = -1                       # one pull that found nobody
    want = brute(x, idx, S, R, w, newcomer)
    got = oracle.segment_aggregate_members(x, idx, S, R, w, newcomer)
    np.testing.assert_allclose(got, want, rtol=0, atol=1e-16)
    got32 = oracle.segment_aggregate_members(x, idx, S, R, w, newcomer, ordered=True)
    assert np.abs(got32 - want).max() <= (2 * R + 3) * 2.0 ** -24 * np.abs(x).max()
    # offline workers keep their model; a newcomer's own values never enter its result
    for v in np.flatnonzero(active == 0):
        assert (got[v] == x[v].astype(np.float64)).all()
    x2 = x.copy()
    x2[newcomer.astype(bool)] = 1e6
    got2 = oracle.segment_aggregate_members(x2, idx, S, R, w, newcomer)
    others_use_newcomer = np.zeros(N, bool)
    for v in range(N):
        others_use_newcomer[v] = np.isin(idx[v], np.flatnonzero(newcomer)).any()
    for v in np.flatnonzero(newcomer):
        if not np.isin(idx[v], np.flatnonzero(newcomer)).any():
            assert (got2[v] == got[v]).all()
