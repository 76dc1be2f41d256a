"""Seeded synthetic inputs for the segmented-gossip round.

This module only draws random tensors; it contains none of the method's
arithmetic (no segmentation, peer choice or averaging), so both the CUDA
path and the CPU checker can be fed from it.

The five workloads mirror the shapes the paper motivates: a small CNN-sized
federation, ResNet-18 / ResNet-50 sized flat vectors and a BERT-large sized
one (the paper quotes 1360 MB for it in its introduction).  Workers hold a
shared base vector plus a small per-worker drift, which is how models that
started from identical parameters (Section 4.1) look after local training.
"""
from __future__ import annotations

import dataclasses

import torch


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    N: int                 # workers
    P: int                 # parameters per worker
    dtype: str             # "f32" or "bf16" storage
    S: int                 # segments
    R: int                 # model replicas (peers per segment)
    rounds: int
    weighted: bool         # per-worker sample counts as |D_j|, else equal
    fused_sgd: bool        # local SGD step fused in front of the aggregation
    sigma_base: float      # std of the shared base vector (0 = no shared base)
    sigma_drift: float     # std of the per-worker part
    sigma_grad: float = 0.0
    lr: float = 0.0
    sampler_seed: int = 1

    def scaled(self, P: int, rounds: int | None = None) -> "Workload":
        """Same structure with a different vector length (for quick checks)."""
        return dataclasses.replace(self, P=P, rounds=self.rounds if rounds is None else rounds,
                                   name="%s@P=%d" % (self.name, P))


WORKLOADS = {
    "cfg1_n8_1m_f32": Workload("cfg1_n8_1m_f32", 8, 1_048_576, "f32", 4, 2, 1, False, False,
                               0.0, 0.05),
    "cfg2_n32_resnet18_f32": Workload("cfg2_n32_resnet18_f32", 32, 11_689_512, "f32", 8, 3, 10,
                                      True, False, 0.05, 0.01),
    "cfg3_n64_resnet50_f32": Workload("cfg3_n64_resnet50_f32", 64, 25_557_032, "f32", 10, 4, 20,
                                      False, False, 0.05, 0.01),
    "cfg4_n128_bf16": Workload("cfg4_n128_bf16", 128, 23_520_842, "bf16", 16, 4, 10, False, False,
                               0.02, 0.005),
    "cfg5_n16_bertlarge_sgd_f32": Workload("cfg5_n16_bertlarge_sgd_f32", 16, 335_141_888, "f32",
                                           32, 4, 5, False, True, 0.02, 0.002, 1e-3, 0.01),
}
WORKLOAD_ORDER = list(WORKLOADS)


def get_workload(key) -> Workload:
    """Look a workload up by name or by 1-based number."""
    if isinstance(key, int) or (isinstance(key, str) and key.isdigit()):
        return WORKLOADS[WORKLOAD_ORDER[int(key) - 1]]
    return WORKLOADS[key]


def _torch_dtype(wl: Workload):
    return torch.float32 if wl.dtype == "f32" else torch.bfloat16


def _gen(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def make_params(wl: Workload, device="cpu", seed: int = 0) -> torch.Tensor:
    """[N][P] parameters: base ~ N(0, sigma_base) shared by all workers (drawn
    from ``seed``) plus N(0, sigma_drift) per worker (drawn from seed+100+w);
    cast to the storage dtype with round-to-nearest-even."""
    dev = torch.device(device)
    out = torch.empty((wl.N, wl.P), dtype=_torch_dtype(wl), device=dev)
    base = None
    if wl.sigma_base > 0.0:
        base = torch.randn(wl.P, generator=_gen(dev, seed), device=dev,
                           dtype=torch.float32) * wl.sigma_base
    for w in range(wl.N):
        row = torch.randn(wl.P, generator=_gen(dev, seed + 100 + w), device=dev,
                          dtype=torch.float32) * wl.sigma_drift
        if base is not None:
            row += base
        out[w].copy_(row)
    return out


def make_grads(wl: Workload, rnd: int, device="cpu", seed: int = 1000) -> torch.Tensor:
    """[N][P] gradients ~ N(0, sigma_grad) for round ``rnd`` (fp32)."""
    dev = torch.device(device)
    out = torch.empty((wl.N, wl.P), dtype=torch.float32, device=dev)
    g = _gen(dev, seed + rnd)
    for w in range(wl.N):
        out[w].copy_(torch.randn(wl.P, generator=g, device=dev, dtype=torch.float32)
                     * wl.sigma_grad)
    return out


def make_weights(wl: Workload, device="cpu", seed: int = 2):
    """|D_j|: integer sample counts uniform in [500, 1500] as fp32, or None
    when every worker holds the same amount of data."""
    if not wl.weighted:
        return None
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    counts = torch.randint(500, 1501, (wl.N,), generator=g, dtype=torch.int64)
    return counts.to(torch.float32).to(device)
