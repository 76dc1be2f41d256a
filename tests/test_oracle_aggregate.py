"""Pins for the oracle's segment-wise aggregation (Eq. 1, Eq. 3, Eq. 4).

Eq. 3 is an exact definition, so it is pinned by exact rational arithmetic
(written a second, different way: per output element, with Python sets and
fractions), by a hand-worked example, and by the special cases the paper
names: S = 1 is plain gossip, R = n-1 is the all-reduce / FedAvg mean.
"""
import json
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def bf16_bits(a):
    """float32 array -> bf16 bit patterns by truncation of exactly representable values."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    assert ((u & 0xFFFF) == 0).all()
    return (u >> 16).astype(np.uint16)


def bf16_to_f64(b):
    return (b.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def brute_force(x, idx, S, R, weights=None, grads=None, lr=0.0):
    """Eq. 3 per output element in exact rationals; P_l as a Python set."""
    N, P = x.shape
    L = -(-P // S)
    out = [[None] * P for _ in range(N)]
    for i in range(N):
        for p in range(P):
            l = p // L
            providers = {i} | {int(j) for j in (idx[i][l] if R else [])}
            assert len(providers) == R + 1
            num = Fraction(0)
            den = Fraction(0)
            for j in providers:
                D = Fraction(float(weights[j])) if weights is not None else Fraction(1)
                v = Fraction(float(x[j, p]))
                if grads is not None:
                    v -= Fraction(float(lr)) * Fraction(float(grads[j, p]))
                num += D * v
                den += D
            out[i][p] = num / den
    return out


# ---------------------------------------------------------------- Eq. 1
def test_segment_bounds_closed_form_and_partition():
    for P in list(range(1, 40)) + [1000, 1_048_576, 11_689_512, 25_557_032, 23_520_842]:
        for S in (1, 2, 3, 4, 7, 8, 10, 16, 32):
            lo, hi = oracle.segment_bounds(P, S)
            L = -(-P // S)
            assert lo[0] == 0 and hi[-1] == P
            assert (lo[1:] == hi[:-1]).all()                 # non-overlapping, no gap
            lens = hi - lo
            assert lens.max() == L and (lens >= 0).all()
            full = lens[lens > 0]
            assert (full[:-1] == L).all()                    # only the tail is shorter
    lo, hi = oracle.segment_bounds(25_557_032, 10)
    assert (hi - lo).tolist() == [2_555_704] * 9 + [2_555_696]
    lo, hi = oracle.segment_bounds(23_520_842, 16)
    assert (hi - lo).tolist() == [1_470_053] * 15 + [1_470_047]
    lo, hi = oracle.segment_bounds(5, 4)                     # L = 2: last segment empty
    assert (hi - lo).tolist() == [2, 2, 1, 0]


# ---------------------------------------------------------------- Eq. 3 / Eq. 4
def test_hand_worked_example():
    g = json.load(open(os.path.join(GOLDEN, "eq3_hand_example.json")))
    x = np.array(g["x"], dtype=np.float32)
    idx = np.array(g["idx"], dtype=np.int32)
    w = np.array(g["weights"], dtype=np.float32)
    want = np.array([[float(Fraction(s)) for s in row] for row in g["expected"]])
    got = oracle.segment_aggregate(x, idx, g["S"], g["R"], weights=w)
    np.testing.assert_allclose(got, want, rtol=4e-16, atol=0)
    got32 = oracle.segment_aggregate_ordered_f32(x, idx, g["S"], g["R"], weights=w)
    np.testing.assert_allclose(got32, want, rtol=3e-7, atol=0)
    # entries whose quotient is a dyadic rational are exact in binary32
    assert got32[0, 0] == 2.0 and got32[0, 1] == 2.0 and got32[1, 2] == 5.0 and got32[1, 3] == 1.0


TINY = [(N, P, S, R) for N in (1, 2, 3, 4, 6) for P in (1, 2, 5, 12, 37)
        for S in (1, 2, 3, 5, 9) for R in range(0, 6) if R <= N - 1 and S <= max(P, 1) + 3]


@pytest.mark.parametrize("N,P,S,R", TINY[::3])
def test_brute_force_exact_rationals(N, P, S, R):
    rng = np.random.default_rng(N * 1000 + P * 10 + S + R)
    x = rng.normal(0, 0.05, (N, P)).astype(np.float32)
    wts = rng.integers(500, 1501, N).astype(np.float32)
    idx = oracle.select_peers(5, 1, N, S, R)
    for weights in (None, wts):
        exact = brute_force(x, idx, S, R, weights)
        got = oracle.segment_aggregate(x, idx, S, R, weights=weights)
        got32 = oracle.segment_aggregate_ordered_f32(x, idx, S, R, weights=weights)
        scale = float(np.abs(x).max())
        for i in range(N):
            for p in range(P):
                e = float(exact[i][p])
                assert abs(got[i, p] - e) <= 4e-16 * scale * (R + 1)
                # binary32 rounding budget: (2R+3) roundings of at most 2^-24 each
                assert abs(float(got32[i, p]) - e) <= (2 * R + 3) * 2.0 ** -24 * scale


def test_brute_force_with_local_step():
    rng = np.random.default_rng(3)
    N, P, S, R = 5, 23, 4, 2
    x = rng.normal(0, 0.02, (N, P)).astype(np.float32)
    g = rng.normal(0, 1e-3, (N, P)).astype(np.float32)
    lr = np.float32(0.01)
    idx = oracle.select_peers(1, 0, N, S, R)
    exact = brute_force(x, idx, S, R, None, g, lr)
    got = oracle.segment_aggregate(x, idx, S, R, grads=g, lr=float(lr))
    got32 = oracle.segment_aggregate_ordered_f32(x, idx, S, R, grads=g, lr=float(lr))
    scale = float(np.abs(x).max())
    want = np.array([[float(v) for v in row] for row in exact])
    assert np.abs(got - want).max() <= 1e-15 * scale
    assert np.abs(got32 - want).max() <= (2 * R + 4) * 2.0 ** -24 * scale
    # fused = "step every worker's model, then aggregate the stepped models"
    # (peers send their locally updated parameters, Section 4.1 steps 1 and 3)
    stepped = (x.astype(np.float64) - float(lr) * g.astype(np.float64))
    two_pass = np.zeros_like(stepped)
    L = -(-P // S)
    for i in range(N):
        for p in range(P):
            prov = [i] + idx[i, p // L].tolist()
            two_pass[i, p] = stepped[prov, p].mean()
    np.testing.assert_allclose(got, two_pass, rtol=0, atol=1e-15)
    # a wrong reading (only the worker's own row stepped) must differ
    own_only = np.zeros_like(stepped)
    for i in range(N):
        for p in range(P):
            prov = idx[i, p // L].tolist()
            own_only[i, p] = (stepped[i, p] + x[prov, p].astype(np.float64).sum()) / (R + 1)
    assert np.abs(own_only - got).max() > 1e-7


def test_ordered_f32_step_equals_two_passes():
    rng = np.random.default_rng(8)
    N, P, S, R = 6, 50, 3, 3
    x = rng.normal(0, 0.02, (N, P)).astype(np.float32)
    g = rng.normal(0, 1e-3, (N, P)).astype(np.float32)
    lr = 0.01
    idx = oracle.select_peers(2, 0, N, S, R)
    fused = oracle.segment_aggregate_ordered_f32(x, idx, S, R, grads=g, lr=lr)
    # numpy has no fma; the product lr*g is exact in binary64 and the sum of two
    # binary64 numbers rounded once to binary64 then to binary32 can double-round,
    # so compare to tolerance of one ulp instead of bits here ...
    stepped = (x.astype(np.float64) - np.float64(np.float32(lr)) * g.astype(np.float64))
    s32 = stepped.astype(np.float32)
    plain = oracle.segment_aggregate_ordered_f32(s32, idx, S, R)
    assert np.abs(fused.astype(np.float64) - plain).max() <= 2.0 ** -23 * np.abs(x).max()


def test_R0_is_identity_bit_exact():
    rng = np.random.default_rng(0)
    x = rng.normal(0, 0.05, (4, 33)).astype(np.float32)
    wts = np.array([3, 5, 7, 11], dtype=np.float32)
    for weights in (None, wts):
        got = oracle.segment_aggregate(x, None, 3, 0, weights=weights)
        assert (got == x.astype(np.float64)).all()
        got32 = oracle.segment_aggregate_ordered_f32(x, None, 3, 0, weights=weights)
        assert (got32.view(np.uint32) == x.view(np.uint32)).all()


@pytest.mark.parametrize("N", [2, 5, 16])
def test_R_full_is_allreduce_mean(N):
    # R = n-1: every worker aggregates all external models and gets the global
    # weighted mean, the FedAvg / all-reduce result (Section 4.3 discussion).
    rng = np.random.default_rng(N)
    P, S = 40, 4
    x = rng.normal(0, 0.05, (N, P)).astype(np.float32)
    wts = rng.integers(500, 1501, N).astype(np.float32)
    idx = oracle.select_peers(1, 0, N, S, N - 1)
    for weights in (None, wts):
        mean = np.average(x.astype(np.float64), axis=0, weights=weights)
        got = oracle.segment_aggregate(x, idx, S, N - 1, weights=weights)
        np.testing.assert_allclose(got, np.broadcast_to(mean, (N, P)), rtol=0, atol=1e-16 * N)
        got32 = oracle.segment_aggregate_ordered_f32(x, idx, S, N - 1, weights=weights)
        assert np.abs(got32 - mean).max() <= (2 * N + 1) * 2.0 ** -24 * np.abs(x).max()


def test_S1_is_plain_gossip_averaging():
    # S = 1: whole models are pulled (naive gossip); no segment logic needed.
    rng = np.random.default_rng(4)
    N, P, R = 7, 29, 2
    x = rng.normal(0, 0.05, (N, P)).astype(np.float32)
    idx = oracle.select_peers(1, 0, N, 1, R)
    got = oracle.segment_aggregate(x, idx, 1, R)
    for i in range(N):
        prov = [i] + idx[i, 0].tolist()
        np.testing.assert_allclose(got[i], x[prov].astype(np.float64).mean(axis=0),
                                   rtol=0, atol=1e-16)


def test_segments_use_their_own_peers():
    # worker j holds the constant vector j: the output of worker i on segment l
    # is then the weighted mean of the provider ids of (i, l) and nothing else.
    N, P, S, R = 9, 41, 5, 3
    x = np.repeat(np.arange(N, dtype=np.float32)[:, None], P, axis=1)
    wts = np.arange(1, N + 1, dtype=np.float32)
    idx = oracle.select_peers(3, 2, N, S, R)
    got = oracle.segment_aggregate(x, idx, S, R, weights=wts)
    lo, hi = oracle.segment_bounds(P, S)
    for i in range(N):
        for l in range(S):
            prov = [i] + idx[i, l].tolist()
            want = sum(float(wts[j]) * j for j in prov) / sum(float(wts[j]) for j in prov)
            assert np.abs(got[i, lo[l]:hi[l]] - want).max() < 1e-14


def test_convexity_and_identical_inputs_and_consensus():
    rng = np.random.default_rng(6)
    N, P, S, R = 8, 64, 4, 2
    x = rng.normal(0, 0.05, (N, P)).astype(np.float32)
    wts = rng.integers(500, 1501, N).astype(np.float32)
    idx = oracle.select_peers(1, 0, N, S, R)
    got = oracle.segment_aggregate(x, idx, S, R, weights=wts)
    assert (got <= x.max(axis=0) + 1e-16).all() and (got >= x.min(axis=0) - 1e-16).all()
    same = np.repeat(x[:1], N, axis=0).copy()
    got_same = oracle.segment_aggregate(same, idx, S, R, weights=wts)
    np.testing.assert_allclose(got_same, same.astype(np.float64), rtol=3e-16, atol=0)
    # repeated rounds without local updates: the per-column spread never grows
    cur = x
    spread = cur.max(axis=0) - cur.min(axis=0)
    for rnd in range(6):
        nxt = oracle.segment_aggregate(cur, oracle.select_peers(1, rnd, N, S, R), S, R,
                                       weights=wts).astype(np.float32)
        s2 = nxt.max(axis=0) - nxt.min(axis=0)
        assert (s2 <= spread + 1e-7).all()
        cur, spread = nxt, s2


def test_column_ranges_are_independent():
    rng = np.random.default_rng(9)
    N, P, S, R = 6, 101, 7, 2
    x = rng.normal(0, 0.05, (N, P)).astype(np.float32)
    idx = oracle.select_peers(1, 0, N, S, R)
    full = oracle.segment_aggregate(x, idx, S, R)
    full32 = oracle.segment_aggregate_ordered_f32(x, idx, S, R)
    for a, b in ((0, 17), (13, 64), (60, 101), (30, 30)):
        slab = np.ascontiguousarray(x[:, a:b])
        part = oracle.segment_aggregate(slab, idx, S, R, P=P, p_begin=a, p_end=b)
        assert (part == full[:, a:b]).all()
        part32 = oracle.segment_aggregate_ordered_f32(slab, idx, S, R, P=P, p_begin=a, p_end=b)
        assert (part32 == full32[:, a:b]).all()


# ---------------------------------------------------------------- bf16 storage
def test_bf16_rounding_rule():
    # round-to-nearest-even on the 16 dropped bits
    def f(u):
        return np.array([u], dtype=np.uint32).view(np.float32)[0]
    assert oracle.f32_to_bf16_rne(f(0x3F800000)) == 0x3F80
    assert oracle.f32_to_bf16_rne(f(0x3F808000)) == 0x3F80      # tie -> even (down)
    assert oracle.f32_to_bf16_rne(f(0x3F818000)) == 0x3F82      # tie -> even (up)
    assert oracle.f32_to_bf16_rne(f(0x3F808001)) == 0x3F81      # above tie
    assert oracle.f32_to_bf16_rne(f(0x3F807FFF)) == 0x3F80      # below tie
    assert oracle.f32_to_bf16_rne(f(0xBF808001)) == 0xBF81
    rng = np.random.default_rng(1)
    v = rng.normal(0, 0.02, 2000).astype(np.float32)
    import torch
    want = torch.from_numpy(v).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = np.array([oracle.f32_to_bf16_rne(float(t)) for t in v], dtype=np.uint16)
    assert (got == want).all()


def test_bf16_storage_matches_exact_within_one_ulp():
    rng = np.random.default_rng(2)
    N, P, S, R = 6, 48, 4, 3
    import torch
    xb = torch.from_numpy(rng.normal(0, 0.02, (N, P)).astype(np.float32)).to(torch.bfloat16)
    bits = xb.view(torch.int16).numpy().view(np.uint16).copy()
    idx = oracle.select_peers(1, 0, N, S, R)
    exact = oracle.segment_aggregate(bits, idx, S, R)
    brute = brute_force(bf16_to_f64(bits).astype(np.float32), idx, S, R)
    want = np.array([[float(v) for v in row] for row in brute])
    assert np.abs(exact - want).max() <= 1e-17
    got = oracle.segment_aggregate_ordered_f32(bits, idx, S, R)
    ulp = 2.0 ** (np.floor(np.log2(np.abs(exact) + 1e-300)) - 7)
    assert (np.abs(bf16_to_f64(got) - exact) <= 0.5 * ulp * (1 + 1e-3)).all()


def test_ordered_f32_is_eq3_as_written():
    # Eq. 3 in binary32, in the fixed order: num = D_self*x_self, num = fma(D_j, x_j, num),
    # den summed in the same order, out = num * (1/den).  With unit weights the products are
    # exact, so num is the plain sequential sum, which numpy's binary32 adds reproduce.
    rng = np.random.default_rng(21)
    N, P, S, R = 7, 41, 3, 4
    x = rng.normal(0, 0.05, (N, P)).astype(np.float32)
    idx = oracle.select_peers(4, 2, N, S, R)
    got = oracle.segment_aggregate_ordered_f32(x, idx, S, R)
    L = -(-P // S)
    rcp = np.float32(1.0) / np.float32(R + 1)
    for i in range(N):
        for p in range(P):
            acc = x[i, p]
            for k in idx[i, p // L]:
                acc = np.float32(acc + x[k, p])
            assert got[i, p] == np.float32(acc * rcp)
    # unit weights given explicitly are the same computation, bit for bit
    ones = np.ones(N, np.float32)
    assert (oracle.segment_aggregate_ordered_f32(x, idx, S, R, weights=ones).view(np.uint32)
            == got.view(np.uint32)).all()
