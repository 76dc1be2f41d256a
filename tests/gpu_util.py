"""Helpers shared by the GPU parity tests: run the CUDA library through its
C ABI binding and compare with the CPU oracle on the same bytes."""
from __future__ import annotations

import numpy as np
import torch

import oracle
import paper_1908_07782_b200 as combo

DEV = "cuda:0"


def to_bits(t: torch.Tensor) -> np.ndarray:
    """Host numpy view the oracle understands: float32, or uint16 for bf16."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def bf16_ulp(v: np.ndarray) -> np.ndarray:
    """Spacing of bf16 numbers (8 significant bits) around |v|, normal range."""
    a = np.maximum(np.abs(v), 2.0 ** -126)
    return 2.0 ** (np.floor(np.log2(a)) - 7)


def gpu_select(seed, rnd, N, S, R):
    idx = torch.full((N, S, max(R, 0)), -7, dtype=torch.int32, device=DEV)
    combo.combo_select_peers(seed, rnd, N, S, R, idx)
    return idx


def gpu_aggregate(x, idx, S, R, weights=None, grads=None, lr=0.0, path=combo.PATH_AUTO,
                  guard=64):
    """Runs the matching C entry point; the output sits inside a larger buffer
    with sentinel words before and after it, which are checked."""
    N, P = x.shape
    combo.combo_set_kernel_path(path)
    try:
        buf = torch.empty(N * P + 2 * guard, dtype=x.dtype, device=x.device)
        sentinel = 1234.5 if x.dtype == torch.float32 else 1232.0
        buf.fill_(sentinel)
        out = buf[guard:guard + N * P].view(N, P)
        assert out.data_ptr() % 16 == 0
        if x.dtype == torch.bfloat16:
            assert grads is None
            combo.combo_segment_aggregate_bf16(x, out, weights, idx, N, P, S, R)
        elif grads is not None:
            combo.combo_segment_aggregate_sgd(x, grads, lr, out, weights, idx, N, P, S, R)
        else:
            combo.combo_segment_aggregate(x, out, weights, idx, N, P, S, R)
        torch.cuda.synchronize()
        used = combo.combo_last_kernel_path()
        assert (buf[:guard] == sentinel).all() and (buf[guard + N * P:] == sentinel).all(), \
            "write outside the output array"
        return out.clone(), used
    finally:
        combo.combo_set_kernel_path(combo.PATH_AUTO)


def check_against_oracle(x, out, idx_np, S, R, weights=None, grads=None, lr=0.0, P=None,
                         p_begin=0, expect_ordered_exact=True):
    """x, out: tensors [N][width] holding columns [p_begin, p_begin+width) of a
    P-vector.  Asserts the tolerance of the library contract against the
    binary64 oracle, and bit equality with the fixed-order binary32 form."""
    xb = to_bits(x)
    gb = to_bits(grads) if grads is not None else None
    wn = weights.detach().cpu().numpy() if weights is not None else None
    lr32 = float(np.float32(lr))
    width = xb.shape[1]
    exact = oracle.segment_aggregate(xb, idx_np, S, R, weights=wn, grads=gb, lr=lr32, P=P,
                                     p_begin=p_begin, p_end=p_begin + width)
    ordered = oracle.segment_aggregate_ordered_f32(xb, idx_np, S, R, weights=wn, grads=gb, lr=lr32,
                                                   P=P, p_begin=p_begin, p_end=p_begin + width)
    got = to_bits(out)
    if x.dtype == torch.bfloat16:
        got64 = bf16_bits_to_f64(got)
        scale = float(np.abs(bf16_bits_to_f64(xb)).max()) if xb.size else 0.0
        # The stored value is RNE_bf16 of a binary32 accumulation: half a bf16 ulp from
        # the rounding plus the binary32 budget d = 1e-6 * max|param| of the accumulate
        # (which dominates only where providers cancel to a value far below max|param|).
        # For values of ordinary size this is tighter than the one-ulp contract.
        d = max(1e-6, (2 * R + 3) * 2.0 ** -24) * scale
        bound = 0.5 * bf16_ulp(np.abs(exact) + d) + d
        assert (np.abs(got64 - exact) <= bound).all(), "bf16 result outside half an ulp + fp32 budget"
        big = np.abs(exact) >= 2.0 ** 9 * d
        assert (np.abs(got64 - exact)[big] <= bf16_ulp(exact)[big]).all(), "bf16 result off by > 1 ulp"
    else:
        scale = float(np.abs(xb).max()) if xb.size else 0.0
        err = float(np.abs(got.astype(np.float64) - exact).max()) if xb.size else 0.0
        # tolerance of the library contract: max |err| <= 1e-6 * max |param|.  It covers
        # the (2R+3) binary32 roundings of the fixed order for R <= 6; beyond that the
        # rounding budget itself, (2R+3) * 2^-24, is the bound.
        tol = max(1e-6, (2 * R + 3 + (1 if grads is not None else 0)) * 2.0 ** -24)
        assert err <= tol * scale, "fp32 result off by %g (scale %g)" % (err, scale)
    if expect_ordered_exact:
        same = (got.view(np.uint16 if x.dtype == torch.bfloat16 else np.uint32) ==
                ordered.view(np.uint16 if x.dtype == torch.bfloat16 else np.uint32))
        assert same.all(), "differs from the fixed-order binary32 form in %d places" % (~same).sum()
    return exact
