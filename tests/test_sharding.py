"""Host side of the worker-sharded round: who hosts whom, what crosses which link
(Section 3: a worker pulls S*R segments, one model's worth per replica)."""
import numpy as np
import pytest

import oracle
from paper_1908_07782_b200 import sharding


@pytest.mark.parametrize("N,world", [(8, 1), (8, 2), (30, 4), (31, 4), (128, 8), (9, 8)])
def test_worker_ranges_partition_the_workers(N, world):
    seen = []
    sizes = []
    for r in range(world):
        a, b = sharding.worker_range(r, world, N)
        sizes.append(b - a)
        seen += list(range(a, b))
        for w in range(a, b):
            assert sharding.owner_of(w, world, N) == r
    assert seen == list(range(N))
    assert max(sizes) - min(sizes) <= 1


@pytest.mark.parametrize("P,S", [(40, 4), (25_557_032, 10), (7, 9), (23_520_842, 16)])
def test_segment_lengths_follow_the_oracle_bounds(P, S):
    lens = sharding.segment_lengths(P, S)
    lo, hi = oracle.segment_bounds(P, S)
    assert (lens == np.asarray(hi) - np.asarray(lo)).all()
    assert lens.sum() == P


def test_pull_traffic_counts_every_pulled_segment_once():
    N, S, R, P, world, e = 32, 8, 3, 11_689_512, 4, 4
    idx = oracle.select_peers(1, 0, N, S, R)
    t = sharding.pull_traffic(idx, world, P, e)
    # every worker pulls R whole models' worth of segments (Section 3, "Model Replica")
    assert t.sum() == N * R * P * e
    for a in range(world):
        lo, hi = sharding.worker_range(a, world, N)
        assert t[a].sum() == (hi - lo) * R * P * e
    # brute force over the table for one pair of ranks
    lens = sharding.segment_lengths(P, S) * e
    want = 0
    for w in range(*sharding.worker_range(1, world, N)):
        for l in range(S):
            for k in idx[w, l]:
                if sharding.owner_of(int(k), world, N) == 3:
                    want += lens[l]
    assert t[1, 3] == want


def test_one_rank_pulls_nothing_over_the_links():
    idx = oracle.select_peers(1, 0, 8, 4, 2)
    t = sharding.pull_traffic(idx, 1, 1_048_576, 4)
    assert t.shape == (1, 1) and t[0, 0] == 8 * 2 * 1_048_576 * 4


def test_row_address_table_for_uneven_shares():
    # every worker's address = its owner's base + its local row; checked against an
    # independent walk over the ranks' ranges, for shares that differ by one
    for N, world in ((7, 3), (10, 4), (64, 8), (9, 9), (13, 2), (5, 1)):
        pitch_bytes = 4096 + 16 * world
        bases = [(g + 1) * (1 << 32) + 256 * g for g in range(world)]
        got = sharding.row_addresses(bases, N, pitch_bytes)
        want = [None] * N
        for g in range(world):
            a, b = sharding.worker_range(g, world, N)
            for local, w in enumerate(range(a, b)):
                assert sharding.owner_of(w, world, N) == g
                want[w] = bases[g] + local * pitch_bytes
        assert got == want
        assert len(set(got)) == N
        sizes = [sharding.worker_range(g, world, N) for g in range(world)]
        assert max(b - a for a, b in sizes) - min(b - a for a, b in sizes) <= 1


def test_distinct_rows_read_counts_shared_pulls_once():
    # two hosted workers that pull the same (peer, segment) share one copy; a hosted worker
    # pulled by another hosted worker costs nothing extra
    N, S, R, P, world = 6, 2, 2, 1000, 3
    idx = np.array([[[2, 4], [1, 5]], [[2, 4], [0, 3]], [[0, 1], [0, 1]], [[0, 1], [0, 1]],
                    [[0, 1], [0, 1]], [[0, 1], [0, 1]]], dtype=np.int32)
    local, remote = sharding.distinct_rows_read(idx, world, 0, P)       # rank 0 hosts workers 0, 1
    # segment 0: pulled {2, 4} (both remote, shared by workers 0 and 1) -> 2 hosted + 2 remote
    # segment 1: worker 0 pulls {1, 5}, worker 1 pulls {0, 3}: 1 and 0 are hosted -> remote {3, 5}
    assert local == pytest.approx(2.0) and remote == pytest.approx(2.0)
    # against the per-pull count of the paper: 2 workers x 2 pulls = 4 rows' worth per segment
    t = sharding.pull_traffic(idx, world, P, 4)
    assert t[0].sum() == 4 * 2 * (P // S) * 4
    # one rank hosting everybody reads every row once
    local, remote = sharding.distinct_rows_read(idx, 1, 0, P)
    assert remote == 0.0 and local == pytest.approx(6.0)
