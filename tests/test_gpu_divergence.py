"""Parity of combo_aggregation_divergence (Eq. 7) with the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
import paper_1908_07782_b200 as combo

from gpu_util import DEV, to_bits

pytestmark = pytest.mark.gpu

# Tolerance.  Deviations d = x - mean are formed in binary32: each carries an absolute error of
# about 2^-24 * |x| from the mean (N fused multiply-adds, random signs) and from the
# subtraction, i.e. a relative error e = 2^-23 * |x| / |d| per term; the squares are summed in
# binary64, so rho inherits at most e (systematic case), far less when the errors average
# out.  The inputs below have |d| >= |x| / 10, hence e <= 1.2e-6; 5e-6 is asserted.
RTOL = 5e-6


def run(models, mean_of, weights, path=combo.PATH_AUTO):
    N, P = models.shape
    e = models.element_size()
    rho = torch.full((N,), -1.0, dtype=torch.float64, device=DEV)
    scratch = torch.empty(combo.combo_divergence_scratch_bytes(N) // 8, dtype=torch.float64, device=DEV)
    scratch.fill_(float("nan"))                      # the call must not rely on its contents
    combo.combo_set_kernel_path(path)
    try:
        combo.combo_aggregation_divergence(models, mean_of, e, weights, N, P, rho, scratch)
        torch.cuda.synchronize()
        used = combo.combo_last_kernel_path()
    finally:
        combo.combo_set_kernel_path(combo.PATH_AUTO)
    return rho.cpu().numpy(), used


def make(N, P, dtype, seed):
    g = torch.Generator().manual_seed(seed)
    base = torch.randn(P, generator=g) * 0.05
    x = (base + torch.randn(N, P, generator=g) * 0.01).to(dtype).to(DEV)
    y = (base + torch.randn(N, P, generator=g) * 0.01).to(dtype).to(DEV)
    w = torch.randint(500, 1501, (N,), generator=g).float().to(DEV)
    return x, y, w


CASES = [
    (8, 100_000, torch.float32), (32, 65_536, torch.float32), (64, 40_004, torch.float32),
    (128, 30_008, torch.bfloat16), (16, 70_000, torch.bfloat16), (1, 5_000, torch.float32),
    (3, 1_000, torch.float32),                    # tiny: fallback kernel
    (7, 100_001, torch.float32),                  # rows only 4-byte aligned: staged per row class
    (40, 50_002, torch.bfloat16),                 # the same for bf16 (pitch = 4 mod 16 bytes)
    (128, 20_010, torch.bfloat16),
    (9, 100_001, torch.bfloat16),                 # odd bf16 pitch: fallback kernel
    (64, 30_000, torch.float32),                  # two arrays of 64 rows: half-width tiles
    (200, 20_000, torch.float32),                 # too many rows for two staged tiles: fallback
    (300, 4_096, torch.bfloat16),                 # more than 256 workers
    (16, 1_500_004, torch.float32),               # few rows: tiles of two boxes, several per CTA, ragged end
    (4, 700_012, torch.bfloat16),                 # tiles of four boxes
]


@pytest.mark.parametrize("N,P,dtype", CASES)
def test_divergence_matches_oracle(N, P, dtype):
    x, y, w = make(N, P, dtype, N + P)
    for weights in (None, w):
        wn = weights.cpu().numpy() if weights is not None else None
        got, _ = run(x, None, weights)
        want = oracle.divergence(to_bits(x), wn)
        np.testing.assert_allclose(got, want, rtol=RTOL, atol=1e-12)
        got, _ = run(x, y, weights)
        want = oracle.divergence(to_bits(x), wn, mean_of=to_bits(y))
        np.testing.assert_allclose(got, want, rtol=RTOL, atol=1e-12)


def test_both_kernels_agree_and_paths_are_taken():
    x, y, w = make(32, 200_000, torch.float32, 5)
    a, used_a = run(x, y, w, combo.PATH_AUTO)
    b, used_b = run(x, y, w, combo.PATH_DIRECT)
    assert used_a == combo.PATH_STAGED and used_b == combo.PATH_DIRECT
    np.testing.assert_allclose(a, b, rtol=RTOL)


def test_round_with_all_replicas_has_no_divergence():
    # R = n-1 leaves no divergence at all (Section 4.3); fewer replicas leave more
    N, P, S = 12, 120_000, 6
    x, _, w = make(N, P, torch.float32, 9)
    means = []
    for R in (1, 3, N - 1):
        idx = torch.empty((N, S, R), dtype=torch.int32, device=DEV)
        combo.combo_select_peers(1, 0, N, S, R, idx)
        out = torch.empty_like(x)
        combo.combo_segment_aggregate(x, out, w, idx, N, P, S, R)
        rho, _ = run(out, x, w)
        means.append(rho.mean())
    assert means[0] > means[1] > 100 * means[2]
    assert means[2] <= 2e-6 * float(torch.linalg.vector_norm(x[0]))


def test_divergence_argument_errors():
    x = torch.zeros(4, 1000, device=DEV)
    rho = torch.zeros(4, dtype=torch.float64, device=DEV)
    small = torch.zeros(8, dtype=torch.float64, device=DEV)
    with pytest.raises(combo.ComboError) as e:
        combo.combo_aggregation_divergence(x, None, 4, None, 4, 1000, rho, small)
    assert e.value.status == 1                     # scratch too small
    big = torch.zeros(combo.combo_divergence_scratch_bytes(4) // 8, dtype=torch.float64, device=DEV)
    with pytest.raises(combo.ComboError):
        combo.combo_aggregation_divergence(x, None, 3, None, 4, 1000, rho, big)
    with pytest.raises(combo.ComboError):
        combo.combo_aggregation_divergence(x, None, 4, None, 0, 1000, rho, big)
