"""The five full-size workloads, run the way the benchmark runs them (peer
selection + aggregation per round, ping-pong buffers, automatic kernel
choice), checked on sampled column ranges.

Eq. 3 couples workers only at equal column, so the oracle can be evaluated on
any set of columns on its own, round after round: the sampled slabs are copied
to the host before each launch and evolved there by the oracle.  Samples cover
every segment boundary, the first and last columns, tile edges and a few
random places.  In addition, where device memory allows, every round is repeated with the
direct-gather kernel (itself pinned to the oracle on slabs of every size) into a third buffer
and the two outputs are compared over the WHOLE array, bit for bit: a tile handed to the wrong
stage at full size would show there even if it missed every sampled span."""
import numpy as np
import pytest
import torch

import oracle
import paper_1908_07782_b200 as combo
from paper_1908_07782_b200 import synth

from gpu_util import DEV, bf16_bits_to_f64, bf16_ulp, to_bits

pytestmark = pytest.mark.gpu


def sample_ranges(wl, rng):
    P, S = wl.P, wl.S
    L = -(-P // S)
    spans = [(0, 300), (P - 300, P)]
    for l in range(1, S):
        b = min(l * L, P)
        spans.append((max(b - 70, 0), min(b + 70, P)))
    for T in (248, 252, 256, 512, 1024, 2048):
        j = int(rng.integers(1, max(P // T, 2)))
        spans.append((max(j * T - 20, 0), min(j * T + 20, P)))
    for _ in range(6):
        a = int(rng.integers(0, P - 256))
        spans.append((a, a + 256))
    return sorted(set(spans))


@pytest.mark.parametrize("name", synth.WORKLOAD_ORDER)
def test_workload_full_size_sampled(name):
    wl = synth.WORKLOADS[name]
    free, _ = torch.cuda.mem_get_info()
    e = 4 if wl.dtype == "f32" else 2
    need = wl.N * wl.P * (2 * e + (4 if wl.fused_sgd else 0)) * 1.1 + 2e9
    if free < need:
        pytest.skip("needs %.0f GB of free device memory" % (need / 1e9))
    whole_array = free >= need + wl.N * wl.P * e * 1.05      # room for the direct kernel's output
    rng = np.random.default_rng(7)
    spans = sample_ranges(wl, rng)
    cur = synth.make_params(wl, DEV)
    nxt = torch.empty_like(cur)
    third = torch.empty_like(cur) if whole_array else None
    weights = synth.make_weights(wl, DEV)
    wn = weights.cpu().numpy() if weights is not None else None
    idx = torch.empty((wl.N, wl.S, wl.R), dtype=torch.int32, device=DEV)
    lr32 = float(np.float32(wl.lr))
    # host copies of the sampled slabs, evolved by the fixed-order binary32 oracle
    chain = {sp: to_bits(cur[:, sp[0]:sp[1]]) for sp in spans}
    scale = float(cur.abs().max())
    for t in range(wl.rounds):
        grads = synth.make_grads(wl, t, DEV) if wl.fused_sgd else None
        combo.combo_select_peers(wl.sampler_seed, t, wl.N, wl.S, wl.R, idx)
        idx_np = oracle.select_peers(wl.sampler_seed, t, wl.N, wl.S, wl.R)
        assert (idx.cpu().numpy() == idx_np).all()
        before = {sp: to_bits(cur[:, sp[0]:sp[1]]) for sp in spans}
        gsl = {sp: to_bits(grads[:, sp[0]:sp[1]]) for sp in spans} if grads is not None else None
        if wl.dtype == "bf16":
            combo.combo_segment_aggregate_bf16(cur, nxt, weights, idx, wl.N, wl.P, wl.S, wl.R)
        elif wl.fused_sgd:
            combo.combo_segment_aggregate_sgd(cur, grads, wl.lr, nxt, weights, idx, wl.N, wl.P, wl.S, wl.R)
        else:
            combo.combo_segment_aggregate(cur, nxt, weights, idx, wl.N, wl.P, wl.S, wl.R)
        torch.cuda.synchronize()
        assert combo.combo_last_kernel_path() in (combo.PATH_STAGED, combo.PATH_TILE)
        if third is not None:
            combo.combo_set_kernel_path(combo.PATH_DIRECT)
            try:
                if wl.dtype == "bf16":
                    combo.combo_segment_aggregate_bf16(cur, third, weights, idx, wl.N, wl.P, wl.S, wl.R)
                elif wl.fused_sgd:
                    combo.combo_segment_aggregate_sgd(cur, grads, wl.lr, third, weights, idx, wl.N, wl.P, wl.S, wl.R)
                else:
                    combo.combo_segment_aggregate(cur, third, weights, idx, wl.N, wl.P, wl.S, wl.R)
            finally:
                combo.combo_set_kernel_path(combo.PATH_AUTO)
            torch.cuda.synchronize()
            assert combo.combo_last_kernel_path() == combo.PATH_DIRECT
            assert torch.equal(nxt, third), (name, t, "staged and direct outputs differ somewhere in the array")
        for sp in spans:
            a, b = sp
            got = to_bits(nxt[:, a:b])
            g = gsl[sp] if gsl is not None else None
            # (i) this round, from the same device inputs, against Eq. 3 in binary64
            exact = oracle.segment_aggregate(before[sp], idx_np, wl.S, wl.R, weights=wn, grads=g, lr=lr32,
                                             P=wl.P, p_begin=a, p_end=b)
            if wl.dtype == "bf16":
                d = 1e-6 * scale
                got64 = bf16_bits_to_f64(got)
                assert (np.abs(got64 - exact) <= 0.5 * bf16_ulp(np.abs(exact) + d) + d).all(), (name, t, sp)
            else:
                assert np.abs(got.astype(np.float64) - exact).max() <= 1e-6 * scale, (name, t, sp)
            # (ii) the chained state, bit for bit against the fixed-order binary32 form
            assert (before[sp].view(np.uint8) == chain[sp].view(np.uint8)).all(), (name, t, sp)
            chain[sp] = oracle.segment_aggregate_ordered_f32(chain[sp], idx_np, wl.S, wl.R, weights=wn, grads=g,
                                                             lr=lr32, P=wl.P, p_begin=a, p_end=b)
            assert (got.view(np.uint8) == chain[sp].view(np.uint8)).all(), (name, t, sp)
        cur, nxt = nxt, cur
        del grads
    combo.combo_device_status()
