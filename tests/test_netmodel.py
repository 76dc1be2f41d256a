"""The paper's network model (Section 5.1) applied to peer tables: closed forms and the
qualitative statements of Section 5.2 ("Benefit of Model Segments")."""
import numpy as np

import oracle
from paper_1908_07782_b200 import netmodel

B = 8e6 * 8          # an 8 MB model, in bits


def test_single_pull_runs_at_the_pair_limit():
    idx = np.array([[[1]], [[0]]], dtype=np.int32)            # two workers pull each other's model
    t, per = netmodel.sync_time(idx, B)
    assert abs(t - B / 10e6) < 1e-9 * t and np.allclose(per, t)


def test_ingress_limit_binds_when_many_segments_arrive():
    # worker 0 pulls 20 segments from 20 different peers: 20 x 10 Mbps > its 100 Mbps
    N, S = 21, 20
    idx = np.full((N, S, 1), -1, dtype=np.int32)
    idx[0, :, 0] = np.arange(1, 21)
    t, per = netmodel.sync_time(idx, B)
    assert abs(t - B / 100e6) < 1e-9 * t and per[1:].max() == 0.0


def test_egress_limit_binds_on_a_popular_sender():
    # 20 workers pull the whole model of worker 0
    N = 21
    idx = np.zeros((N, 1, 1), dtype=np.int32)
    idx[0, 0, 0] = -1
    t, _ = netmodel.sync_time(idx, B)
    assert abs(t - B / (100e6 / 20)) < 1e-9 * t


def test_two_segments_from_one_peer_share_the_pair_link():
    idx = np.array([[[1], [1]], [[-1], [-1]]], dtype=np.int32)
    t, _ = netmodel.sync_time(idx, B)
    assert abs(t - B / 10e6) < 1e-9 * t


def test_rebalancing_after_a_transfer_ends():
    # worker 0 pulls half the model from each of 11 peers (S = 2 would need 2 rows; use sizes):
    # 11 flows share 100 Mbps (9.09 each) although the pair links allow 10
    N = 12
    idx = np.full((N, 11, 1), -1, dtype=np.int32)
    idx[0, :, 0] = np.arange(1, 12)
    t, _ = netmodel.sync_time(idx, B)
    assert abs(t - B / 100e6) < 1e-9 * t


def test_segments_halve_the_sync_time_until_the_worker_limit_is_reached():
    # 30 workers, R = 2 (the paper's setting): S = 2 halves the time of S = 1, and from
    # S * R * 10 Mbps >= 100 Mbps on, more segments no longer help
    N, R = 30, 2
    times = {}
    for S in range(1, 11):
        ts = [netmodel.sync_time(oracle.select_peers(seed, 0, N, S, R), B)[0] for seed in range(5)]
        times[S] = float(np.median(ts))
    assert abs(times[2] / times[1] - 0.5) < 0.08
    assert times[1] > times[2] > times[3] > times[4]
    floor = R * B / 100e6                                # R models through a 100 Mbps port
    for S in range(6, 11):
        assert floor <= times[S] < 1.7 * floor
    assert max(times[S] for S in range(6, 11)) / min(times[S] for S in range(6, 11)) < 1.35
    assert times[1] > 3.0 * times[6]


def test_more_replicas_cost_proportionally_more_once_saturated():
    N, S = 30, 10
    t2 = np.median([netmodel.sync_time(oracle.select_peers(s, 0, N, S, 2), B)[0] for s in range(5)])
    t4 = np.median([netmodel.sync_time(oracle.select_peers(s, 0, N, S, 4), B)[0] for s in range(5)])
    assert 1.6 < t4 / t2 < 2.6
