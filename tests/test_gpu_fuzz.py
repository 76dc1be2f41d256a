"""Randomised shapes: the aggregation kernels against the oracle and each other."""
import numpy as np
import pytest
import torch

import oracle
import paper_1908_07782_b200 as combo

from gpu_util import DEV, check_against_oracle, gpu_aggregate

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("seed", range(24))
def test_random_shapes(seed):
    rng = np.random.default_rng(1000 + seed)
    dtype = torch.float32 if rng.random() < 0.6 else torch.bfloat16
    N = int(rng.choice([2, 3, 5, 8, 13, 16, 31, 32, 48, 64, 96, 128, 160]))
    R = int(rng.integers(0, min(N - 1, 17) + 1))
    S = int(rng.choice([1, 2, 3, 4, 7, 8, 10, 16, 32]))
    P = int(rng.integers(20_000, 400_000 // max(N // 16, 1)))
    P += int(rng.integers(0, 16))                       # every alignment residue
    fused = dtype == torch.float32 and rng.random() < 0.4
    weighted = rng.random() < 0.5
    g = torch.Generator().manual_seed(seed)
    x = (torch.randn(N, P, generator=g) * 0.05).to(dtype).to(DEV)
    grads = (torch.randn(N, P, generator=g) * 1e-3).to(DEV) if fused else None
    w = torch.randint(500, 1501, (N,), generator=g).float().to(DEV) if weighted else None
    idx_np = oracle.select_peers(seed, seed % 5, N, S, R)
    idx = torch.from_numpy(idx_np).to(DEV) if R > 0 else None
    a, _ = gpu_aggregate(x, idx, S, R, weights=w, grads=grads, lr=0.01, path=combo.PATH_STAGED)
    b, _ = gpu_aggregate(x, idx, S, R, weights=w, grads=grads, lr=0.01, path=combo.PATH_DIRECT)
    assert torch.equal(a, b), (N, P, S, R, dtype, fused)
    c, _ = gpu_aggregate(x, idx, S, R, weights=w, grads=grads, lr=0.01, path=combo.PATH_TILE)
    assert torch.equal(a, c), (N, P, S, R, dtype, fused)
    lo, hi = 0, min(P, 3000)
    mid = P // 2
    for (c0, c1) in ((lo, hi), (max(mid - 1500, 0), min(mid + 1500, P)), (max(P - 3000, 0), P)):
        check_against_oracle(x[:, c0:c1].contiguous(), a[:, c0:c1].contiguous(), idx_np, S, R, weights=w,
                             grads=grads[:, c0:c1].contiguous() if fused else None, lr=0.01, P=P, p_begin=c0)
    combo.combo_device_status()


@pytest.mark.parametrize("seed", range(10))
def test_random_long_rows(seed):
    # few rows, long vectors: tens of tiles per CTA, so that most tiles come from the
    # dispenser, with every alignment residue and segment boundaries inside tiles
    rng = np.random.default_rng(5000 + seed)
    dtype = torch.float32 if rng.random() < 0.6 else torch.bfloat16
    N = int(rng.choice([2, 4, 5, 8, 12, 16, 24]))
    R = int(rng.integers(1, min(N - 1, 6) + 1))
    S = int(rng.choice([1, 3, 4, 7, 10, 32]))
    P = int(rng.integers(1_000_000, 3_000_000)) + int(rng.integers(0, 16))
    fused = dtype == torch.float32 and rng.random() < 0.4
    weighted = rng.random() < 0.5
    g = torch.Generator().manual_seed(seed)
    x = (torch.randn(N, P, generator=g) * 0.05).to(dtype).to(DEV)
    grads = (torch.randn(N, P, generator=g) * 1e-3).to(DEV) if fused else None
    w = torch.randint(500, 1501, (N,), generator=g).float().to(DEV) if weighted else None
    idx_np = oracle.select_peers(seed, 3, N, S, R)
    idx = torch.from_numpy(idx_np).to(DEV)
    a, used = gpu_aggregate(x, idx, S, R, weights=w, grads=grads, lr=0.01, path=combo.PATH_STAGED)
    assert used == combo.PATH_STAGED, (N, P, S, R, dtype, fused)
    b, _ = gpu_aggregate(x, idx, S, R, weights=w, grads=grads, lr=0.01, path=combo.PATH_DIRECT)
    assert torch.equal(a, b), (N, P, S, R, dtype, fused)
    c, used_c = gpu_aggregate(x, idx, S, R, weights=w, grads=grads, lr=0.01, path=combo.PATH_TILE)
    assert torch.equal(a, c), (N, P, S, R, dtype, fused)
    if (P * x.element_size()) % 16 == 0:
        assert used_c == combo.PATH_TILE
    L = -(-P // S)
    windows = [(0, 2000), (max(P - 2000, 0), P)]
    if S > 1:
        windows.append((L - 1000, min(L + 1000, P)))        # across the first segment boundary
    for (c0, c1) in windows:
        check_against_oracle(x[:, c0:c1].contiguous(), a[:, c0:c1].contiguous(), idx_np, S, R, weights=w,
                             grads=grads[:, c0:c1].contiguous() if fused else None, lr=0.01, P=P, p_begin=c0)
    combo.combo_device_status()


@pytest.mark.parametrize("N,P,S,R,dtype,weighted", [
    (40, 1_300_004, 10, 4, torch.float32, False),     # 40 KB stages: a ring of four
    (48, 1_250_000, 7, 3, torch.float32, True),       # 48 KB stages: a ring of three
    (80, 1_300_008, 16, 4, torch.bfloat16, False),    # aligned bf16 rows, 40 KB stages
    (100, 1_300_002, 16, 4, torch.bfloat16, True),    # rows of differing phase, 50 KB stages
    (20, 1_300_000, 5, 2, torch.float32, False),      # with gradients beside the parameters: 40 KB stages
])
def test_long_kernels_with_deeper_rings(N, P, S, R, dtype, weighted):
    # many rows and tens of tiles per CTA: stages below 64 KB, of which the ring holds three or
    # four; whole-array equality with the direct kernel, windows against the oracle
    fused = dtype == torch.float32 and N == 20
    g = torch.Generator().manual_seed(N)
    x = (torch.randn(N, P, generator=g) * 0.05).to(dtype).to(DEV)
    grads = (torch.randn(N, P, generator=g) * 1e-3).to(DEV) if fused else None
    w = torch.randint(500, 1501, (N,), generator=g).float().to(DEV) if weighted else None
    idx_np = oracle.select_peers(N, 2, N, S, R)
    idx = torch.from_numpy(idx_np).to(DEV)
    a, used = gpu_aggregate(x, idx, S, R, weights=w, grads=grads, lr=0.01)
    assert used == combo.PATH_STAGED
    b, _ = gpu_aggregate(x, idx, S, R, weights=w, grads=grads, lr=0.01, path=combo.PATH_DIRECT)
    assert torch.equal(a, b), (N, P, S, R, dtype)
    L = -(-P // S)
    for (c0, c1) in ((0, 1500), (L - 700, L + 700), (P - 1500, P)):
        check_against_oracle(x[:, c0:c1].contiguous(), a[:, c0:c1].contiguous(), idx_np, S, R, weights=w,
                             grads=grads[:, c0:c1].contiguous() if fused else None, lr=0.01, P=P, p_begin=c0)
    combo.combo_device_status()
