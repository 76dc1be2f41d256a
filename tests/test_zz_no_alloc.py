"""combo_aggregation_divergence_noalloc: the entry point for callers that cannot
allocate device memory (its partial sums live in a fixed array inside the
library).  It must give what combo_aggregation_divergence gives with caller
scratch, call after call, although all calls share that one array and the
array keeps the previous call's contents.

This file is collected last on purpose, so that a run that stops at the first
failure has already been through every other test."""
import numpy as np
import pytest
import torch

import oracle
import paper_1908_07782_b200 as combo

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
RTOL = 5e-6          # the tolerance the divergence parity tests use


def reference(models, mean_of, weights):
    N, P = models.shape
    rho = torch.empty(N, dtype=torch.float64, device=DEV)
    scratch = torch.empty(combo.combo_divergence_scratch_bytes(N) // 8, dtype=torch.float64, device=DEV)
    combo.combo_aggregation_divergence(models, mean_of, models.element_size(), weights, N, P, rho, scratch)
    torch.cuda.synchronize()
    return rho.cpu().numpy()


def no_alloc(models, mean_of, weights):
    N, P = models.shape
    rho = torch.full((N,), -1.0, dtype=torch.float64, device=DEV)
    combo.combo_aggregation_divergence_noalloc(models, mean_of, models.element_size(), weights, N, P, rho)
    torch.cuda.synchronize()
    return rho.cpu().numpy()


def oracle_rho(models, mean_of, weights):
    """Eq. 7 by the CPU oracle on the same bytes."""
    def bits(t):
        t = t.detach().cpu().contiguous()
        return t.view(torch.int16).numpy().view(np.uint16) if t.dtype == torch.bfloat16 else t.numpy()
    return oracle.divergence(bits(models), weights.cpu().numpy(), mean_of=None if mean_of is None else bits(mean_of))


def inputs(N, P, dtype, seed):
    g = torch.Generator().manual_seed(seed)
    base = torch.randn(P, generator=g) * 0.05
    x = (base + torch.randn(N, P, generator=g) * 0.01).to(dtype).to(DEV)
    y = (base + torch.randn(N, P, generator=g) * 0.01).to(dtype).to(DEV)
    w = torch.randint(500, 1501, (N,), generator=g).float().to(DEV)
    return x, y, w


def test_two_calls_in_a_row_match_the_scratch_taking_entry_point():
    # first a large call that fills much of the fixed array, then a smaller one of another
    # shape and type: stale partial sums of the first must not leak into the second
    first = inputs(128, 60_000, torch.float32, 1)
    second = inputs(24, 200_000, torch.bfloat16, 2)
    for x, y, w in (first, second):
        want = reference(x, y, w)
        got = no_alloc(x, y, w)
        assert (got >= 0).all()
        np.testing.assert_allclose(got, want, rtol=RTOL, atol=1e-12)
        # and directly against the oracle, not only through the other entry point
        np.testing.assert_allclose(got, oracle_rho(x, y, w), rtol=RTOL, atol=1e-12)
    # and once more on the fallback kernel (rows not 16-byte aligned), against its own mean
    x, _, w = inputs(9, 50_001, torch.float32, 3)
    got = no_alloc(x, None, w)
    np.testing.assert_allclose(got, reference(x, None, w), rtol=RTOL, atol=1e-12)
    np.testing.assert_allclose(got, oracle_rho(x, None, w), rtol=RTOL, atol=1e-12)
    combo.combo_device_status()


def test_more_workers_than_the_fixed_array_holds_is_refused():
    x, _, _ = inputs(129, 1_000, torch.float32, 4)
    rho = torch.zeros(129, dtype=torch.float64, device=DEV)
    with pytest.raises(combo.ComboError) as e:
        combo.combo_aggregation_divergence_noalloc(x, None, 4, None, 129, 1_000, rho)
    assert e.value.status == 6
    assert "128" in combo.load().combo_last_cuda_error().decode()
