"""Pins for the oracle's peer sampler (Section 4.1 step 2) and its generator.

The paper fixes no random generator, so the exact tables are unpinned by it;
what it does fix are properties: targets are OTHER workers, drawn without
replacement until none is left, requests spread evenly, and all segments come
from different workers when S*R fits into the pool.  The generator itself is
pinned to the published splitmix64 sequence.
"""
import collections
import itertools
import json
import os

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def test_splitmix64_published_sequence():
    want = [int(s) for s in open(os.path.join(GOLDEN, "splitmix64_seed1234567.txt"))
            if s.strip() and not s.startswith("#")]
    assert oracle.splitmix64_stream(1234567, len(want)) == want


def test_rand32_first_link_is_splitmix_of_seed():
    # With round = w = e = t = 0 the xor-ed counter words vanish, so rand32 is
    # three plain splitmix64 steps, each restarted from the previous output.
    for seed in (0, 1, 1234567, 2**64 - 1):
        h = oracle.splitmix64_stream(seed, 1)[0]
        h = oracle.splitmix64_stream(h, 1)[0]
        h = oracle.splitmix64_stream(h, 1)[0]
        assert oracle.rand32(seed, 0, 0, 0, 0) == h >> 32


def test_rand32_depends_on_every_field():
    base = (11, 3, 5, 2, 9)
    ref = oracle.rand32(*base)
    flips = []
    for pos in range(5):
        for bit in range(0, 32, 5):
            args = list(base)
            args[pos] ^= (1 << bit)
            v = oracle.rand32(*args)
            assert v != ref
            flips.append(bin(v ^ ref).count("1"))
    assert 13.0 < np.mean(flips) < 19.0      # avalanche: about half of 32 bits


def test_rand32_is_uniform_enough():
    vals = np.array([oracle.rand32(5, r, w, 0, t) for r in range(20) for w in range(20)
                     for t in range(1, 26)], dtype=np.uint64)
    assert abs(vals.mean() / 2**32 - 0.5) < 0.01
    hist = np.bincount((vals >> np.uint64(28)).astype(np.int64), minlength=16)
    exp = len(vals) / 16
    chi2 = ((hist - exp) ** 2 / exp).sum()
    assert chi2 < 45.0                         # 15 dof, p ~ 1e-4


CASES = [(N, S, R) for N in (2, 3, 4, 5, 8, 16, 33) for S in (1, 2, 4, 7, 16)
         for R in (0, 1, 2, 3, 4, 7, 32) if R <= N - 1]


@pytest.mark.parametrize("N,S,R", CASES)
def test_sampler_invariants(N, S, R):
    for seed, rnd in ((1, 0), (1, 1), (99, 7)):
        idx = oracle.select_peers(seed, rnd, N, S, R)
        assert idx.shape == (N, S, R) and idx.dtype == np.int32
        if R == 0:
            continue
        assert idx.min() >= 0 and idx.max() < N
        for w in range(N):
            assert not (idx[w] == w).any()                       # never the worker itself
            for l in range(S):
                row = idx[w, l]
                assert (np.diff(row) > 0).all()                  # ascending => distinct
            flat = idx[w].ravel()
            if S * R <= N - 1:                                   # all from different workers
                assert len(set(flat.tolist())) == S * R
            use = np.bincount(flat, minlength=N)
            others = np.delete(use, w)
            assert others.max() - others.min() <= 1              # requests spread evenly
            assert others.sum() == S * R


def test_sampler_is_a_pure_function_of_its_counter():
    a = oracle.select_peers(1, 4, 16, 8, 3)
    b = oracle.select_peers(1, 4, 16, 8, 3)
    assert (a == b).all()
    assert (oracle.select_peers(1, 5, 16, 8, 3) != a).any()      # round changes the table
    assert (oracle.select_peers(2, 4, 16, 8, 3) != a).any()      # seed changes the table
    # workers draw independently: worker 3's rows do not depend on N's other rows' count
    assert not (a[3] == a[4]).all()


def test_sampler_rejects_bad_arguments():
    for N, S, R in ((0, 1, 0), (4, 0, 1), (4, 2, -1), (4, 2, 4), (1, 1, 1)):
        with pytest.raises(ValueError):
            oracle.select_peers(1, 0, N, S, R)
    assert oracle.select_peers(1, 0, 1, 3, 0).shape == (1, 3, 0)


def test_shuffle_is_uniform_over_permutations():
    # N = 5, R = 1, S = 4: worker 0's four draws are one full epoch, so
    # idx[0, :, 0] is the shuffled order of workers 1..4 itself.
    counts = collections.Counter()
    trials = 24 * 500
    for seed in range(trials):
        idx = oracle.select_peers(seed, 0, 5, 4, 1)
        counts[tuple(idx[0, :, 0].tolist())] += 1
    perms = list(itertools.permutations([1, 2, 3, 4]))
    assert set(counts) == set(perms)
    exp = trials / 24
    chi2 = sum((counts[p] - exp) ** 2 / exp for p in perms)
    assert chi2 < 58.0                         # 23 dof, p ~ 1e-4


def test_shuffle_uniform_across_rounds_and_workers():
    # same statistic, varying round and worker instead of the seed
    counts = collections.Counter()
    n = 0
    for rnd in range(1500):
        idx = oracle.select_peers(3, rnd, 4, 3, 1)
        for w in range(4):
            counts[(w, tuple(idx[w, :, 0].tolist()))] += 1
        n += 1
    for w in range(4):
        others = [v for v in range(4) if v != w]
        chi2 = 0.0
        for p in itertools.permutations(others):
            chi2 += (counts[(w, p)] - n / 6) ** 2 / (n / 6)
        assert chi2 < 27.0                     # 5 dof, p ~ 5e-5


def test_refill_repair_keeps_segment_distinct_and_uniform():
    # N = 4 (pool of 3), R = 2, S = 2: the 4th draw opens a new epoch while the
    # second segment already holds one peer.  That peer must not come again,
    # and the other two must be equally likely.
    pair = collections.Counter()
    for seed in range(6000):
        idx = oracle.select_peers(seed, 0, 4, 2, 2)
        first = set(idx[0, 0].tolist())
        second = idx[0, 1].tolist()
        assert second[0] != second[1]
        left = ({1, 2, 3} - first).pop()       # third draw = last of epoch 0
        assert left in second
        other = (set(second) - {left}).pop()
        pair[(left, other)] += 1
    for left in (1, 2, 3):
        a, b = [pair[(left, o)] for o in (1, 2, 3) if o != left]
        assert abs(a - b) < 5.0 * np.sqrt(a + b) / 2 + 1


def test_first_draw_uniform_over_others():
    hist = np.zeros(8)
    for seed in range(7000):
        hist[oracle.select_peers(seed, 2, 8, 1, 1)[5, 0, 0]] += 1
    assert hist[5] == 0
    exp = 1000.0
    chi2 = ((np.delete(hist, 5) - exp) ** 2 / exp).sum()
    assert chi2 < 30.0                         # 6 dof


def test_regression_tables_match_committed_copy():
    data = json.load(open(os.path.join(GOLDEN, "peer_tables.json")))
    for c in data["cases"]:
        got = oracle.select_peers(c["seed"], c["round"], c["N"], c["S"], c["R"])
        assert got.tolist() == c["idx"]
