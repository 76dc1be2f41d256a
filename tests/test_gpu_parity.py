"""Parity of the CUDA library (through its C ABI) with the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
import paper_1908_07782_b200 as combo
from paper_1908_07782_b200 import synth

pytestmark = pytest.mark.gpu

from gpu_util import DEV, check_against_oracle, gpu_aggregate, gpu_select, to_bits  # noqa: E402


# ------------------------------------------------------------------ peer sampler
SAMPLER_CASES = [
    (8, 4, 2), (32, 8, 3), (64, 10, 4), (128, 16, 4), (16, 32, 4),      # the five workloads
    (2, 1, 1), (2, 5, 1), (3, 7, 2), (4, 2, 2), (5, 4, 1), (5, 9, 4), (9, 3, 8), (33, 2, 32),
    (130, 3, 1), (300, 5, 7), (257, 2, 256), (1000, 2, 999), (4097, 3, 5), (1, 4, 0), (6, 3, 0),
]


@pytest.mark.parametrize("N,S,R", SAMPLER_CASES)
def test_select_peers_bit_exact(N, S, R):
    for seed, rnd in ((1, 0), (1, 7), (0xDEADBEEFCAFEF00D, 4_000_000_000)):
        got = gpu_select(seed, rnd, N, S, R).cpu().numpy()
        want = oracle.select_peers(seed, rnd, N, S, R)
        assert got.shape == want.shape
        assert (got == want).all()


def test_select_peers_default_stream_entry():
    idx = torch.zeros((8, 4, 2), dtype=torch.int32, device=DEV)
    combo.combo_select_peers_default_stream(1, 0, 8, 4, 2, idx)
    torch.cuda.synchronize()
    assert (idx.cpu().numpy() == oracle.select_peers(1, 0, 8, 4, 2)).all()


def test_select_peers_rounds_of_every_workload():
    for name, wl in synth.WORKLOADS.items():
        for rnd in range(wl.rounds):
            got = gpu_select(wl.sampler_seed, rnd, wl.N, wl.S, wl.R).cpu().numpy()
            assert (got == oracle.select_peers(wl.sampler_seed, rnd, wl.N, wl.S, wl.R)).all(), name


def test_validate_idx():
    N, S, R = 16, 4, 3
    idx = gpu_select(1, 0, N, S, R)
    flag = torch.full((1,), 99, dtype=torch.int32, device=DEV)
    combo.combo_validate_idx(idx, N, S, R, flag)
    assert int(flag.item()) == 0
    for pos, val in ((5, 0), (7, N), (9, -1)):
        bad = idx.clone().view(-1)
        if pos == 5:
            bad[pos] = pos // (S * R)          # the worker itself
        else:
            bad[pos] = val
        combo.combo_validate_idx(bad, N, S, R, flag)
        assert int(flag.item()) != 0
    bad = idx.clone()
    bad[3, 2, 1] = bad[3, 2, 0]                # repeated peer
    combo.combo_validate_idx(bad, N, S, R, flag)
    assert int(flag.item()) != 0


# ------------------------------------------------------------------ aggregation, small sweep
def _inputs(N, P, dtype, seed, sigma=0.05):
    g = torch.Generator(device="cpu").manual_seed(seed)
    x = (torch.randn(N, P, generator=g) * sigma).to(dtype).to(DEV)
    grads = (torch.randn(N, P, generator=g) * 1e-3).to(DEV)
    counts = torch.randint(500, 1501, (N,), generator=g).float().to(DEV)
    return x, grads, counts


SMALL = [(N, P, S, R) for N in (1, 2, 3, 5, 8) for P in (1, 2, 3, 7, 8, 9, 31, 64, 70, 257)
         for S in (1, 2, 3, 9) for R in (0, 1, 2, 4, 7) if R <= N - 1]


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_aggregate_tiny_shapes_exhaustive(dtype):
    # every small P (odd alignments, P < S with empty segments), both kernels where they apply
    for (N, P, S, R) in SMALL:
        x, grads, counts = _inputs(N, P, dtype, N * 131 + P)
        idx_np = oracle.select_peers(3, 1, N, S, R)
        idx = torch.from_numpy(idx_np).to(DEV)
        for weights in (None, counts):
            out, used = gpu_aggregate(x, idx, S, R, weights=weights)
            assert used == combo.PATH_DIRECT
            check_against_oracle(x, out, idx_np, S, R, weights=weights)
        if dtype == torch.float32:
            out, _ = gpu_aggregate(x, idx, S, R, grads=grads, lr=0.01)
            check_against_oracle(x, out, idx_np, S, R, grads=grads, lr=0.01)


MEDIUM = [
    # N, P, S, R, dtype, weighted
    (8, 40_000, 4, 2, torch.float32, False),
    (8, 40_001, 4, 2, torch.float32, True),       # rows not 16-byte aligned (fp32, granule 4)
    (32, 20_003, 8, 3, torch.float32, True),
    (32, 20_004, 8, 3, torch.float32, True),      # odd segment length, aligned rows
    (64, 9_992, 10, 4, torch.float32, False),     # last segment shorter
    (16, 33_000, 32, 4, torch.float32, False),
    (5, 50_000, 3, 4, torch.float32, True),       # R = N-1
    (12, 30_000, 5, 8, torch.float32, True),      # largest R of the narrow unspecialised kernel
    (12, 30_000, 5, 9, torch.float32, True),      # the wide one
    (20, 30_000, 10, 16, torch.float32, True),    # largest R the staged kernel takes (Section 5.2 sweeps R to 16)
    (20, 30_002, 10, 16, torch.bfloat16, False),  # the same with differing row phases
    (20, 30_000, 3, 17, torch.float32, True),     # beyond it: direct kernel
    (7, 30_000, 3, 0, torch.float32, False),      # R = 0
    (1, 30_000, 3, 0, torch.float32, False),      # a single worker
    (128, 5_002, 16, 4, torch.bfloat16, False),   # row pitch = 4 mod 16 bytes (granule 4)
    (128, 5_003, 16, 4, torch.bfloat16, True),    # odd pitch (granule 2)
    (128, 5_120, 16, 4, torch.bfloat16, False),   # aligned rows
    (20, 20_000, 7, 3, torch.bfloat16, True),
    (9, 70_001, 2, 2, torch.bfloat16, False),
    (256, 3_000, 4, 4, torch.float32, False),     # so many rows that a stage holds 256-byte row pieces
    (230, 3_004, 2, 4, torch.float32, True),
    (250, 4_000, 3, 2, torch.bfloat16, False),    # the same in bf16 (128-column boxes)
    (140, 6_000, 3, 3, torch.float32, True),      # 512-byte row pieces
    (30, 40_000, 10, 12, torch.float32, True),    # many replicas among few workers: dense evaluation of whole tiles
    (30, 40_000, 10, 16, torch.bfloat16, False),
    (33, 20_000, 3, 9, torch.float32, False),     # a last block of one row
    (32, 20_000, 4, 13, torch.bfloat16, True),
    (34, 20_000, 4, 13, torch.float32, True),     # too many workers for it: the warp-per-row form
]


@pytest.mark.parametrize("N,P,S,R,dtype,weighted", MEDIUM)
@pytest.mark.parametrize("path", [combo.PATH_DIRECT, combo.PATH_STAGED])
def test_aggregate_medium_both_kernels(N, P, S, R, dtype, weighted, path):
    x, grads, counts = _inputs(N, P, dtype, 17 * N + P % 1000)
    weights = counts if weighted else None
    idx_np = oracle.select_peers(1, 2, N, S, R)
    idx = torch.from_numpy(idx_np).to(DEV) if R > 0 else None
    out, used = gpu_aggregate(x, idx, S, R, weights=weights, path=path)
    if path == combo.PATH_STAGED and R <= 16:
        assert used == combo.PATH_STAGED
    check_against_oracle(x, out, idx_np, S, R, weights=weights)
    if R == 0:
        assert torch.equal(out, x)                                   # identity, bit for bit
    if dtype == torch.float32:
        out, _ = gpu_aggregate(x, idx, S, R, weights=weights, grads=grads, lr=0.01, path=path)
        check_against_oracle(x, out, idx_np, S, R, weights=weights, grads=grads, lr=0.01)


@pytest.mark.parametrize("N,P,S,R,dtype,weighted", MEDIUM)
def test_aggregate_medium_one_tile_per_cta(N, P, S, R, dtype, weighted):
    # the kernel for short inputs (one tile per CTA); rows whose 16-byte phases differ and
    # R > 16 fall back to the other kernels, everything else must really run on it
    x, grads, counts = _inputs(N, P, dtype, 17 * N + P % 1000)
    weights = counts if weighted else None
    idx_np = oracle.select_peers(1, 2, N, S, R)
    idx = torch.from_numpy(idx_np).to(DEV) if R > 0 else None
    out, used = gpu_aggregate(x, idx, S, R, weights=weights, path=combo.PATH_TILE)
    if (P * x.element_size()) % 16 == 0 and R <= 16 and N <= 128:
        assert used == combo.PATH_TILE
    check_against_oracle(x, out, idx_np, S, R, weights=weights)
    if dtype == torch.float32:
        out, used = gpu_aggregate(x, idx, S, R, weights=weights, grads=grads, lr=0.01, path=combo.PATH_TILE)
        check_against_oracle(x, out, idx_np, S, R, weights=weights, grads=grads, lr=0.01)


@pytest.mark.parametrize("tile", [256, 512, 1024, 2048])
def test_one_tile_per_cta_tile_widths(tile):
    # several boxes per tile, ragged last tile, segment boundaries inside tiles
    N, P, S, R = 8, 100_004, 7, 3
    x, grads, counts = _inputs(N, P, torch.float32, 5)
    idx_np = oracle.select_peers(9, 0, N, S, R)
    idx = torch.from_numpy(idx_np).to(DEV)
    combo.combo_set_tuning(tile, 0)
    try:
        out, used = gpu_aggregate(x, idx, S, R, weights=counts, path=combo.PATH_TILE)
        assert used == combo.PATH_TILE
        check_against_oracle(x, out, idx_np, S, R, weights=counts)
        out, used = gpu_aggregate(x, idx, S, R, grads=grads, lr=0.01, path=combo.PATH_TILE)
        if tile <= 1024:
            assert used == combo.PATH_TILE
        check_against_oracle(x, out, idx_np, S, R, grads=grads, lr=0.01)
        xb = x[:, :100_000].contiguous().to(torch.bfloat16)      # a 16-byte multiple per row in bf16 too
        outb, used = gpu_aggregate(xb, idx, S, R, path=combo.PATH_TILE)
        assert used == combo.PATH_TILE
        check_against_oracle(xb, outb, idx_np, S, R)
    finally:
        combo.combo_set_tuning(0, 0)


@pytest.mark.parametrize("tile,stages", [(256, 2), (256, 8), (512, 3), (768, 2), (1024, 3), (0, 0)])
def test_staged_tile_shapes(tile, stages):
    # many tiles per CTA, several TMA boxes per tile, ragged last tile, segment
    # boundaries inside tiles
    N, P, S, R = 16, 1_000_004, 6, 3
    x, grads, counts = _inputs(N, P, torch.float32, 5)
    idx_np = oracle.select_peers(9, 0, N, S, R)
    idx = torch.from_numpy(idx_np).to(DEV)
    combo.combo_set_tuning(tile, stages)
    try:
        out, used = gpu_aggregate(x, idx, S, R, weights=counts, path=combo.PATH_STAGED)
        assert used == combo.PATH_STAGED
        check_against_oracle(x, out, idx_np, S, R, weights=counts)
        out, used = gpu_aggregate(x, idx, S, R, weights=counts, grads=grads, lr=0.01, path=combo.PATH_STAGED)
        if tile <= 512:
            assert used == combo.PATH_STAGED
        check_against_oracle(x, out, idx_np, S, R, weights=counts, grads=grads, lr=0.01)
        xb = x[:, :600_016].contiguous().to(torch.bfloat16)
        combo.combo_set_tuning(tile, stages)
        outb, used = gpu_aggregate(xb, idx, S, R, path=combo.PATH_STAGED)
        assert used == combo.PATH_STAGED
        check_against_oracle(xb, outb, idx_np, S, R)
    finally:
        combo.combo_set_tuning(0, 0)


@pytest.mark.parametrize("P,dtype", [(1_000_001, torch.float32), (1_000_002, torch.float32),
                                     (1_000_003, torch.float32), (600_001, torch.bfloat16),
                                     (600_002, torch.bfloat16), (600_004, torch.bfloat16),
                                     (600_006, torch.bfloat16)])
def test_staged_unaligned_rows(P, dtype):
    # row pitches of every residue: 2, 4 or 8 row classes, 4- and 2-byte granules
    N, S, R = 13, 5, 4
    x, grads, counts = _inputs(N, P, dtype, 21)
    idx_np = oracle.select_peers(4, 1, N, S, R)
    idx = torch.from_numpy(idx_np).to(DEV)
    out, used = gpu_aggregate(x, idx, S, R, weights=counts, path=combo.PATH_STAGED)
    assert used == combo.PATH_STAGED
    check_against_oracle(x, out, idx_np, S, R, weights=counts)
    if dtype == torch.float32:
        out, used = gpu_aggregate(x, idx, S, R, grads=grads, lr=0.01, path=combo.PATH_STAGED)
        assert used == combo.PATH_STAGED
        check_against_oracle(x, out, idx_np, S, R, grads=grads, lr=0.01)


@pytest.mark.parametrize("N,P,S,R,dtype", [
    (3, 100_001, 2, 2, torch.bfloat16),     # more row classes (8) than workers
    (2, 100_003, 3, 1, torch.float32),      # two workers, one peer
    (5, 65_537, 1, 4, torch.float32),       # S = 1 (plain gossip), R = n-1
    (6, 70_000, 7, 5, torch.bfloat16),      # R without a specialised kernel
    (200, 3_000, 4, 3, torch.float32),      # many workers, short rows (segments shorter than a tile)
    (130, 40_000, 2, 2, torch.bfloat16),    # more than 128 workers
    (150, 30_000, 4, 3, torch.float32),     # so many binary32 rows that only half-width boxes fit two stages
    (176, 20_004, 3, 4, torch.float32),
    (24, 300_002, 5, 4, torch.bfloat16),    # few rows with differing phases: word-mode tiles of several boxes
    (6, 400_001, 4, 2, torch.float32),      # the same for binary32 (4 row classes)
    (10, 200_003, 3, 3, torch.bfloat16),    # odd bf16 pitch (8 classes, 2-byte granule), several boxes
])
def test_staged_odd_shapes(N, P, S, R, dtype):
    x, grads, counts = _inputs(N, P, dtype, 77)
    idx_np = oracle.select_peers(2, 5, N, S, R)
    idx = torch.from_numpy(idx_np).to(DEV)
    out, used = gpu_aggregate(x, idx, S, R, weights=counts, path=combo.PATH_STAGED)
    check_against_oracle(x, out, idx_np, S, R, weights=counts)
    out2, _ = gpu_aggregate(x, idx, S, R, weights=counts, path=combo.PATH_DIRECT)
    assert torch.equal(out, out2)                 # both kernels follow the same fixed order


def test_special_cases_on_device():
    N, P, S = 6, 100_000, 4
    x, _, counts = _inputs(N, P, torch.float32, 3)
    # R = n-1: every worker gets the global weighted mean (the all-reduce result)
    idx_np = oracle.select_peers(1, 0, N, S, N - 1)
    idx = torch.from_numpy(idx_np).to(DEV)
    for path in (combo.PATH_DIRECT, combo.PATH_STAGED):
        out, _ = gpu_aggregate(x, idx, S, N - 1, weights=counts, path=path)
        mean = np.average(x.cpu().numpy().astype(np.float64), axis=0, weights=counts.cpu().numpy())
        assert np.abs(out.cpu().numpy() - mean).max() <= 1e-6 * float(x.abs().max())
        # identical inputs stay identical
        same = x[:1].repeat(N, 1).contiguous()
        out, _ = gpu_aggregate(same, idx, S, N - 1, weights=counts, path=path)
        assert (out - same).abs().max().item() <= 1e-6 * float(x.abs().max())
        # convexity
        i2 = torch.from_numpy(oracle.select_peers(1, 0, N, S, 2)).to(DEV)
        out, _ = gpu_aggregate(x, i2, S, 2, weights=counts, path=path)
        assert (out <= x.max(dim=0).values + 1e-9).all() and (out >= x.min(dim=0).values - 1e-9).all()


def test_argument_errors():
    N, P, S, R = 4, 1000, 2, 1
    x = torch.zeros(N, P, device=DEV)
    out = torch.zeros(N, P, device=DEV)
    idx = gpu_select(1, 0, N, S, R)
    E = combo.ComboError
    with pytest.raises(E) as e:
        combo.combo_segment_aggregate(x, x, None, idx, N, P, S, R)
    assert e.value.status == 2                                        # alias
    both = torch.zeros(2 * N * P, device=DEV)
    with pytest.raises(E) as e:
        combo.combo_segment_aggregate(both[:N * P], both[N * P - 4:2 * N * P - 4], None, idx, N, P, S, R)
    assert e.value.status == 2                                        # partial overlap
    with pytest.raises(E) as e:
        combo.combo_segment_aggregate(both[1:N * P + 1], out, None, idx, N, P, S, R)
    assert e.value.status == 1                                        # misaligned base
    for bad in ((0, P, S, R), (N, 0, S, R), (N, P, 0, R), (N, P, S, -1), (N, P, S, N)):
        with pytest.raises(E) as e:
            combo.combo_segment_aggregate(x, out, None, idx, *bad)
        assert e.value.status == 1
    with pytest.raises(E) as e:
        combo.combo_segment_aggregate(x, out, None, None, N, P, S, R)
    assert e.value.status == 1                                        # idx required when R > 0
    with pytest.raises(E) as e:
        combo.combo_select_peers(1, 0, 4, 2, 4, idx)
    assert e.value.status == 1
    combo.combo_device_status()


def test_column_shards_need_no_exchange():
    # two shards of the columns, each aggregated on its own, give the full result
    N, P, S, R = 8, 120_000, 5, 2
    x, grads, counts = _inputs(N, P, torch.float32, 11)
    idx_np = oracle.select_peers(1, 0, N, S, R)
    idx = torch.from_numpy(idx_np).to(DEV)
    full, _ = gpu_aggregate(x, idx, S, R, weights=counts)
    cut = 50_004
    for (a, b) in ((0, cut), (cut, P)):
        shard = x[:, a:b].contiguous()
        out = torch.empty_like(shard)
        combo.combo_segment_aggregate_cols(shard, None, 0.0, out, 4, counts, idx, N, P, S, R, a, b - a,
                                           b - a)
        torch.cuda.synchronize()
        assert torch.equal(out, full[:, a:b])
        check_against_oracle(shard, out, idx_np, S, R, weights=counts, P=P, p_begin=a)


def test_round_from_host_memory():
    N, P, S, R = 8, 50_000, 4, 2
    g = torch.Generator().manual_seed(1)
    hx = (torch.randn(N, P, generator=g) * 0.05).pin_memory()
    hw = torch.randint(500, 1501, (N,), generator=g).float()
    hout = torch.empty_like(hx).pin_memory()
    hidx = torch.empty((N, S, R), dtype=torch.int32).pin_memory()
    d_in = torch.empty(N, P, device=DEV)
    d_out = torch.empty(N, P, device=DEV)
    d_w = torch.empty(N, device=DEV)
    d_idx = torch.empty((N, S, R), dtype=torch.int32, device=DEV)
    combo.combo_round_host(hx, None, 0.0, hout, 4, hw, 1, 3, 1, N, P, S, R, d_in, None, d_out, d_w, d_idx,
                           hidx)
    idx_np = oracle.select_peers(1, 3, N, S, R)
    assert (hidx.numpy() == idx_np).all()
    check_against_oracle(hx, hout, idx_np, S, R, weights=hw)
    # three chained rounds: each round's input is the previous round's output
    combo.combo_round_host(hx, None, 0.0, hout, 4, hw, 1, 3, 3, N, P, S, R, d_in, None, d_out, d_w, d_idx,
                           hidx)
    cur = hx.numpy()
    for t in range(3):
        idx_t = oracle.select_peers(1, 3 + t, N, S, R)
        cur = oracle.segment_aggregate_ordered_f32(cur, idx_t, S, R, weights=hw.numpy())
    assert (hidx.numpy() == idx_t).all()
    assert (hout.numpy().view(np.uint32) == cur.view(np.uint32)).all()


@pytest.mark.parametrize("P,fused", [(9_000_004, False), (9_000_001, False), (4_500_000, True)])
def test_round_from_host_memory_in_chunks(P, fused):
    # large enough for several column chunks to be in flight; the result must equal the
    # same rounds run on device-resident buffers, bit for bit
    N, S, R, rounds = 8, 5, 3, 3
    g = torch.Generator().manual_seed(2)
    hx = torch.empty(N, P).pin_memory()
    hx.copy_(torch.randn(N, P, generator=g) * 0.05)
    hg = None
    if fused:
        hg = torch.empty(N, P).pin_memory()
        hg.copy_(torch.randn(N, P, generator=g) * 1e-3)
    hw = torch.randint(500, 1501, (N,), generator=g).float()
    hout = torch.empty_like(hx).pin_memory()
    d_in = torch.empty(N, P, device=DEV)
    d_out = torch.empty(N, P, device=DEV)
    d_g = torch.empty(N, P, device=DEV) if fused else None
    d_w = torch.empty(N, device=DEV)
    d_idx = torch.empty((N, S, R), dtype=torch.int32, device=DEV)
    combo.combo_round_host(hx, hg, 0.01, hout, 4, hw, 5, 0, rounds, N, P, S, R, d_in, d_g, d_out, d_w, d_idx)
    cur = hx.to(DEV)
    nxt = torch.empty_like(cur)
    gd = hg.to(DEV) if fused else None
    wd = hw.to(DEV)
    for t in range(rounds):
        combo.combo_select_peers(5, t, N, S, R, d_idx)
        if fused:
            combo.combo_segment_aggregate_sgd(cur, gd, 0.01, nxt, wd, d_idx, N, P, S, R)
        else:
            combo.combo_segment_aggregate(cur, nxt, wd, d_idx, N, P, S, R)
        cur, nxt = nxt, cur
    torch.cuda.synchronize()
    assert torch.equal(hout.to(DEV), cur)
    # and one sampled slab against the oracle, first round only
    idx0 = oracle.select_peers(5, 0, N, S, R)
    a, b = P // 2 - 100, P // 2 + 100
    combo.combo_round_host(hx, hg, 0.01, hout, 4, hw, 5, 0, 1, N, P, S, R, d_in, d_g, d_out, d_w, d_idx)
    check_against_oracle(hx[:, a:b].contiguous(), hout[:, a:b].contiguous(), idx0, S, R, weights=hw,
                         grads=hg[:, a:b].contiguous() if fused else None, lr=0.01, P=P, p_begin=a)


def test_largest_worker_count():
    # N at the library's limit (COMBO_MAX_WORKERS): sampler bit-exact, aggregation through the
    # direct kernel (too many rows to stage), and one more worker is refused
    N, P, S, R = 8192, 96, 2, 3
    idx = gpu_select(7, 4, N, S, R)
    idx_np = oracle.select_peers(7, 4, N, S, R)
    assert (idx.cpu().numpy() == idx_np).all()
    x, _, counts = _inputs(N, P, torch.float32, 5)
    out, used = gpu_aggregate(x, idx, S, R, weights=counts)
    assert used == combo.PATH_DIRECT
    check_against_oracle(x, out, idx_np, S, R, weights=counts)
    with pytest.raises(combo.ComboError) as e:
        combo.combo_select_peers(7, 4, N + 1, S, R, torch.empty((N + 1, S, R), dtype=torch.int32, device=DEV))
    assert e.value.status == 1


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("path", [combo.PATH_AUTO, combo.PATH_STAGED, combo.PATH_DIRECT])
def test_wide_inputs_run_as_column_shards(dtype, path):
    # inputs wider than one launch takes are cut into column shards inside the call; with the
    # limit lowered to 40,000 columns a 150,001-column input takes four launches, which must
    # give the bits of the single launch (segment boundaries fall inside shards)
    N, P, S, R = 9, 150_001, 4, 3
    x, grads, counts = _inputs(N, P, dtype, 77)
    idx_np = oracle.select_peers(2, 5, N, S, R)
    idx = torch.from_numpy(idx_np).to(DEV)
    whole, _ = gpu_aggregate(x, idx, S, R, weights=counts, path=path)
    combo.combo_set_launch_columns(40_000)
    try:
        cut, _ = gpu_aggregate(x, idx, S, R, weights=counts, path=path)
        assert torch.equal(whole, cut)
        check_against_oracle(x, cut, idx_np, S, R, weights=counts)
        if dtype == torch.float32:
            cut, _ = gpu_aggregate(x, idx, S, R, grads=grads, lr=0.01, path=path)
            check_against_oracle(x, cut, idx_np, S, R, grads=grads, lr=0.01)
    finally:
        combo.combo_set_launch_columns(0)


def test_a_wait_that_runs_out_is_reported_once():
    # the give-up path of the bounded waits: a self-check kernel waits (a thousand polls) on a
    # barrier nothing signals, sets the status word and returns; the context stays usable
    combo.combo_device_status()
    combo.combo_debug_dead_wait()
    with pytest.raises(combo.ComboError) as e:
        combo.combo_device_status()
    assert e.value.status == 5
    assert "site 99" in combo.load().combo_last_cuda_error().decode()
    combo.combo_device_status()                     # cleared: reported once
    # and the library works as before (the dispenser ring was cleaned with the status word)
    N, P, S, R = 8, 300_000, 4, 2
    x, _, counts = _inputs(N, P, torch.float32, 3)
    idx_np = oracle.select_peers(1, 0, N, S, R)
    idx = torch.from_numpy(idx_np).to(DEV)
    for path in (combo.PATH_STAGED, combo.PATH_TILE):
        out, used = gpu_aggregate(x, idx, S, R, weights=counts, path=path)
        assert used == path
        check_against_oracle(x, out, idx_np, S, R, weights=counts)
    combo.combo_device_status()
