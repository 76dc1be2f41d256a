"""Synchronization time of one segmented-gossip round under the paper's network
model (Section 5.1, "Network settings"): a fully connected topology in which
every worker has a maximum bandwidth (100 Mbps in the paper) and every pair of
workers an available bandwidth (10 Mbps).

Host-side model, numpy only.  Input is a peer table ``idx[N][S][R]`` as produced
by ``combo_select_peers``: worker ``w`` pulls segment ``l`` (``1/S`` of the model)
from each ``idx[w][l][r] >= 0``.

Readings (the paper does not spell its simulator out):
  * all pulls of a round start together, when the local updates are done
    (Section 4.1 steps 3 and 4);
  * the per-worker limit applies to what a worker receives and, separately, to
    what it sends; the pair limit applies per direction;
  * concurrent transfers share limits max-min fairly (progressive filling) and
    rates are re-balanced whenever a transfer ends;
  * a worker's synchronization time is when its last pulled segment arrives;
    the round's is the maximum over workers.
"""
from __future__ import annotations

import numpy as np


def sync_time(idx, model_bits: float, node_bps: float = 100e6, pair_bps: float = 10e6):
    """Returns (round_time_s, per_worker_time_s[N]) for one round."""
    idx = np.asarray(idx)
    N, S, R = idx.shape
    seg_bits = model_bits / S
    # one flow per (receiver, sender): segments pulled from the same peer share the pair link
    # and are sent back to back, so they behave as one transfer of their total size
    sizes = {}
    for w in range(N):
        for k in idx[w].ravel():
            if k >= 0:
                sizes[(w, int(k))] = sizes.get((w, int(k)), 0.0) + seg_bits
    flows = list(sizes.keys())
    remaining = np.array([sizes[f] for f in flows], dtype=np.float64)
    recv = np.array([f[0] for f in flows])
    send = np.array([f[1] for f in flows])
    alive = remaining > 0
    finish = np.zeros(len(flows))
    now = 0.0
    while alive.any():
        rate = _max_min_rates(recv, send, alive, N, node_bps, pair_bps)
        dt = np.min(remaining[alive] / rate[alive])
        now += dt
        remaining[alive] -= rate[alive] * dt
        done = alive & (remaining <= 1e-9 * seg_bits)
        finish[done] = now
        alive &= ~done
    per_worker = np.zeros(N)
    for i, (w, _) in enumerate(flows):
        per_worker[w] = max(per_worker[w], finish[i])
    return float(per_worker.max() if len(flows) else 0.0), per_worker


def _max_min_rates(recv, send, alive, N, node_bps, pair_bps):
    """Progressive filling: every unfrozen flow grows at the same speed until a limit
    (its pair link, its receiver's ingress, its sender's egress) is reached."""
    F = len(recv)
    rate = np.zeros(F)
    frozen = ~alive
    cap_in = np.full(N, node_bps, dtype=np.float64)
    cap_out = np.full(N, node_bps, dtype=np.float64)
    head = np.full(F, pair_bps, dtype=np.float64)          # room left on the flow's own pair link
    while not frozen.all():
        live = ~frozen
        n_in = np.bincount(recv[live], minlength=N)
        n_out = np.bincount(send[live], minlength=N)
        with np.errstate(divide="ignore", invalid="ignore"):
            inc_in = np.where(n_in > 0, cap_in / n_in, np.inf)
            inc_out = np.where(n_out > 0, cap_out / n_out, np.inf)
        inc = min(head[live].min(), inc_in.min(), inc_out.min())
        rate[live] += inc
        head[live] -= inc
        cap_in -= inc * n_in
        cap_out -= inc * n_out
        tight_in = (cap_in <= 1e-9 * node_bps) & (n_in > 0)
        tight_out = (cap_out <= 1e-9 * node_bps) & (n_out > 0)
        frozen |= live & ((head <= 1e-9 * pair_bps) | tight_in[recv] | tight_out[send])
    return rate
