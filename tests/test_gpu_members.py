"""Dynamic workers (Section 4.2) on the device: sampling over the online pool and
aggregation without a newcomer's own model, against the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
import paper_1908_07782_b200 as combo

from gpu_util import DEV, bf16_bits_to_f64, bf16_ulp, to_bits

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("N,S,R", [(8, 4, 2), (12, 5, 3), (33, 3, 6), (128, 16, 4), (300, 2, 5), (6, 7, 2)])
def test_select_peers_online_bit_exact(N, S, R):
    rng = np.random.default_rng(N * 7 + S)
    idx = torch.empty((N, S, R), dtype=torch.int32, device=DEV)
    # all online: the same table as the plain sampler
    combo.combo_select_peers_online(3, 1, N, S, R, None, idx)
    assert (idx.cpu().numpy() == oracle.select_peers(3, 1, N, S, R)).all()
    combo.combo_select_peers_online(3, 1, N, S, R, [1] * N, idx)
    assert (idx.cpu().numpy() == oracle.select_peers(3, 1, N, S, R)).all()
    for trial in range(4):
        active = np.ones(N, np.uint8)
        n_off = int(rng.integers(1, max(2, N - R - 1)))
        active[rng.choice(N, size=min(n_off, N - R - 1), replace=False)] = 0
        idx.fill_(-7)
        combo.combo_select_peers_online(trial, 2, N, S, R, active.tolist(), idx)
        want = oracle.select_peers_active(trial, 2, N, S, R, active)
        assert (idx.cpu().numpy() == want).all()
    with pytest.raises(combo.ComboError):
        combo.combo_select_peers_online(1, 0, N, S, R, [1] * R + [0] * (N - R), idx)   # R online in all: R-1 others


CASES = [(8, 40_000, 4, 2, torch.float32), (13, 50_001, 5, 4, torch.float32), (32, 20_004, 8, 3, torch.float32),
         (128, 5_002, 16, 4, torch.bfloat16), (20, 30_000, 3, 6, torch.bfloat16), (6, 3_000, 2, 3, torch.float32),
         (24, 40_000, 4, 10, torch.float32), (30, 24_000, 5, 12, torch.bfloat16)]    # many replicas


# unit weights (no weights array) take kernels of their own for bfloat16 rows: the sum of the
# providers' values by mixed-precision adds, with the provider count in the table entry
CASES_UNIT = [(128, 5_002, 16, 4, torch.bfloat16), (20, 30_000, 3, 6, torch.bfloat16),
              (16, 40_008, 4, 4, torch.bfloat16), (30, 24_000, 5, 12, torch.bfloat16),
              (13, 50_001, 5, 4, torch.float32)]


@pytest.mark.parametrize("N,P,S,R,dtype,weighted", [c + (True,) for c in CASES] + [c + (False,) for c in CASES_UNIT])
@pytest.mark.parametrize("path", [combo.PATH_DIRECT, combo.PATH_STAGED])
def test_aggregate_members(N, P, S, R, dtype, weighted, path):
    rng = np.random.default_rng(N + P)
    g = torch.Generator().manual_seed(N)
    x = (torch.randn(N, P, generator=g) * 0.05 + 0.01).to(dtype)
    w = torch.randint(500, 1501, (N,), generator=g).float()
    active = np.ones(N, np.uint8)
    active[rng.choice(N, size=max(1, (N - R - 1) // 3), replace=False)] = 0
    online = np.flatnonzero(active)
    newcomer = np.zeros(N, np.uint8)
    newcomer[rng.choice(online, size=min(2, len(online) - 1), replace=False)] = 1
    idx_np = oracle.select_peers_active(5, 3, N, S, R, active)
    # nobody pulls from a newcomer (it has no model yet): those pulls found no peer
    for v in range(N):
        idx_np[v][np.isin(idx_np[v], np.flatnonzero(newcomer))] = -1
    veteran = [int(v) for v in online if not newcomer[v]]
    idx_np[veteran[-1], 0, :] = -1                             # a segment with no peer at all
    xb = to_bits(x)
    wn = w.numpy() if weighted else None
    exact = oracle.segment_aggregate_members(xb, idx_np, S, R, wn, newcomer)
    ordered = oracle.segment_aggregate_members(xb, idx_np, S, R, wn, newcomer, ordered=True)
    # on the device the newcomers' rows hold NaN: they must never be read
    xd = x.clone()
    xd[torch.from_numpy(newcomer.astype(bool))] = float("nan")
    xd = xd.to(DEV)
    out = torch.empty_like(xd)
    idx = torch.from_numpy(idx_np).to(DEV)
    combo.combo_set_kernel_path(path)
    try:
        combo.combo_segment_aggregate_members(xd, out, w.to(DEV) if weighted else None, idx, newcomer.tolist(),
                                              N, P, S, R)
        torch.cuda.synchronize()
    finally:
        combo.combo_set_kernel_path(combo.PATH_AUTO)
    got = to_bits(out)
    scale = float(x.float().abs().max())
    if dtype == torch.bfloat16:
        d = 1e-6 * scale
        assert (np.abs(bf16_bits_to_f64(got) - exact) <= 0.5 * bf16_ulp(np.abs(exact) + d) + d).all()
        assert (got == ordered).all()
    else:
        assert np.isfinite(got).all()
        assert np.abs(got.astype(np.float64) - exact).max() <= max(1e-6, (2 * R + 3) * 2.0 ** -24) * scale
        assert (got.view(np.uint32) == ordered.view(np.uint32)).all()
    # offline workers keep their model bit for bit
    for v in np.flatnonzero(active == 0):
        assert (got[v] == xb[v]).all()
    combo.combo_device_status()


@pytest.mark.parametrize("N,P,S,R,dtype", [(24, 60_000, 4, 10, torch.float32), (30, 48_000, 5, 14, torch.bfloat16),
                                           (21, 60_004, 3, 9, torch.float32)])
def test_many_replicas_with_absent_peers_and_no_newcomer(N, P, S, R, dtype):
    # offline workers and pulls that found no peer, but nobody new: with R > 8 among few workers
    # whole tiles are evaluated densely (every staged row meets every output with a coefficient
    # that is zero for non-providers); the bits must still be those of the fixed order
    rng = np.random.default_rng(N + R)
    g = torch.Generator().manual_seed(N)
    x = (torch.randn(N, P, generator=g) * 0.05 + 0.01).to(dtype)
    w = torch.randint(500, 1501, (N,), generator=g).float()
    active = np.ones(N, np.uint8)
    active[rng.choice(N, size=3, replace=False)] = 0
    idx_np = oracle.select_peers_active(6, 2, N, S, R, active)
    online = np.flatnonzero(active)
    idx_np[online[0], 0, :] = -1                       # a segment with no peer at all
    idx_np[online[1], S - 1, R // 2:] = -1             # half the pulls missing
    xb = to_bits(x)
    ordered = oracle.segment_aggregate_members(xb, idx_np, S, R, w.numpy(), np.zeros(N, np.uint8), ordered=True)
    xd = x.to(DEV)
    idx = torch.from_numpy(idx_np).to(DEV)
    outs = []
    for path in (combo.PATH_STAGED, combo.PATH_DIRECT):
        out = torch.empty_like(xd)
        combo.combo_set_kernel_path(path)
        try:
            combo.combo_segment_aggregate_members(xd, out, w.to(DEV), idx, None, N, P, S, R)
            torch.cuda.synchronize()
            assert combo.combo_last_kernel_path() == path
        finally:
            combo.combo_set_kernel_path(combo.PATH_AUTO)
        assert (to_bits(out).view(np.uint8) == ordered.view(np.uint8)).all(), path
        outs.append(out)
    assert torch.equal(outs[0], outs[1])
    combo.combo_device_status()
