"""CPU oracle of the segmented-gossip round: ctypes front of ``combo_oracle.c``.

TEST INFRASTRUCTURE ONLY.  Tests, the smoke check and the benchmark's CPU
baseline import this package; the CUDA library and its Python binding never
do.  The shared object is compiled with gcc on first use (or by ``build()``).

All arithmetic lives in the C file; this module only marshals numpy arrays.
bf16 arrays are passed as ``uint16`` bit patterns.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "combo_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile ``combo_oracle.c`` into ``liboracle.so`` beside it."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _LIB + ".%d.tmp" % os.getpid()
            subprocess.check_call(
                ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-fPIC",
                 "-shared", "-o", tmp, _SRC, "-lm"])
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is not None:
        return _lib
    lib = ctypes.CDLL(build())
    i32p = ctypes.POINTER(ctypes.c_int32)
    i64p = ctypes.POINTER(ctypes.c_int64)
    lib.oracle_segment_length.restype = ctypes.c_int64
    lib.oracle_segment_length.argtypes = [ctypes.c_int64, ctypes.c_int]
    lib.oracle_segment_bounds.restype = None
    lib.oracle_segment_bounds.argtypes = [ctypes.c_int64, ctypes.c_int, i64p, i64p]
    lib.oracle_splitmix64_next.restype = ctypes.c_uint64
    lib.oracle_splitmix64_next.argtypes = [ctypes.POINTER(ctypes.c_uint64)]
    lib.oracle_rand32.restype = ctypes.c_uint32
    lib.oracle_rand32.argtypes = [ctypes.c_uint64, ctypes.c_uint32, ctypes.c_uint32,
                                  ctypes.c_uint32, ctypes.c_uint32]
    lib.oracle_select_peers.restype = ctypes.c_int
    lib.oracle_select_peers.argtypes = [ctypes.c_uint64, ctypes.c_uint32, ctypes.c_int,
                                        ctypes.c_int, ctypes.c_int, i32p]
    lib.oracle_f32_to_bf16_rne.restype = ctypes.c_uint16
    lib.oracle_f32_to_bf16_rne.argtypes = [ctypes.c_float]
    lib.oracle_segment_aggregate.restype = ctypes.c_int
    lib.oracle_segment_aggregate.argtypes = [
        ctypes.c_void_p, ctypes.c_void_p, ctypes.c_double, ctypes.c_int, ctypes.c_int64,
        ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_int,
        ctypes.c_int, ctypes.c_int64, ctypes.c_int64, ctypes.c_void_p]
    lib.oracle_segment_aggregate_ordered_f32.restype = ctypes.c_int
    lib.oracle_segment_aggregate_ordered_f32.argtypes = [
        ctypes.c_void_p, ctypes.c_void_p, ctypes.c_float, ctypes.c_int, ctypes.c_int64,
        ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_int,
        ctypes.c_int, ctypes.c_int64, ctypes.c_int64, ctypes.c_void_p]
    lib.oracle_divergence.restype = ctypes.c_int
    lib.oracle_divergence.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p,
                                      ctypes.c_int, ctypes.c_int64, ctypes.c_void_p]
    lib.oracle_select_peers_active.restype = ctypes.c_int
    lib.oracle_select_peers_active.argtypes = [ctypes.c_uint64, ctypes.c_uint32, ctypes.c_int, ctypes.c_int,
                                               ctypes.c_int, ctypes.c_void_p, i32p]
    lib.oracle_segment_aggregate_members.restype = ctypes.c_int
    lib.oracle_segment_aggregate_members.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p,
                                                     ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int,
                                                     ctypes.c_int64, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                                     ctypes.c_void_p]
    _lib = lib
    return lib


def segment_bounds(P: int, S: int):
    """Eq. 1: (lo, hi) int64 arrays of the S segments of a P-vector."""
    lib = _load()
    lo = np.zeros(S, dtype=np.int64)
    hi = np.zeros(S, dtype=np.int64)
    lib.oracle_segment_bounds(P, S, lo.ctypes.data_as(ctypes.POINTER(ctypes.c_int64)),
                              hi.ctypes.data_as(ctypes.POINTER(ctypes.c_int64)))
    return lo, hi


def splitmix64_stream(seed: int, count: int):
    """The first ``count`` outputs of splitmix64 started from state ``seed``."""
    lib = _load()
    state = ctypes.c_uint64(seed)
    return [int(lib.oracle_splitmix64_next(ctypes.byref(state))) for _ in range(count)]


def rand32(seed: int, rnd: int, w: int, e: int, t: int) -> int:
    return int(_load().oracle_rand32(seed, rnd, w, e, t))


def f32_to_bf16_rne(x: float) -> int:
    return int(_load().oracle_f32_to_bf16_rne(x))


def select_peers(seed: int, rnd: int, N: int, S: int, R: int) -> np.ndarray:
    """Section 4.1 step (2): peer table int32 [N][S][R], rows ascending."""
    lib = _load()
    idx = np.zeros((N, S, max(R, 0)), dtype=np.int32)
    rc = lib.oracle_select_peers(seed, rnd, N, S, R,
                                 idx.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)))
    if rc != 0:
        raise ValueError("oracle_select_peers: invalid arguments")
    return idx


def _slab(a: np.ndarray, elem: int):
    want = np.float32 if elem == 4 else np.uint16
    if a.dtype != want or a.ndim != 2 or not a.flags.c_contiguous:
        raise ValueError("expected C-contiguous 2-D %s array" % np.dtype(want).name)
    return a.ctypes.data, a.shape[1]


def _common(x, grads, weights, idx, P, S, R, p_begin, p_end):
    elem = 4 if x.dtype == np.float32 else 2
    xptr, pitch = _slab(x, elem)
    N = x.shape[0]
    if P is None:
        P = pitch
    if p_end is None:
        p_end = p_begin + pitch
    if p_end - p_begin > pitch:
        raise ValueError("column range wider than the slab")
    gptr = None
    if grads is not None:
        gptr, gp = _slab(grads, elem)
        if gp != pitch or grads.shape[0] != N:
            raise ValueError("grads shape mismatch")
    wptr = None
    if weights is not None:
        weights = np.ascontiguousarray(weights, dtype=np.float32)
        if weights.shape != (N,):
            raise ValueError("weights shape mismatch")
        wptr = weights.ctypes.data
    iptr = None
    if R > 0:
        idx = np.ascontiguousarray(idx, dtype=np.int32)
        if idx.shape != (N, S, R):
            raise ValueError("idx shape mismatch")
        iptr = idx.ctypes.data
    return elem, xptr, pitch, gptr, wptr, iptr, N, P, p_begin, p_end, (weights, idx)


def segment_aggregate(x, idx, S, R, weights=None, grads=None, lr=0.0, P=None,
                      p_begin=0, p_end=None) -> np.ndarray:
    """Eq. 3 + Eq. 4 in binary64.  ``x`` is float32 or uint16(bf16) [N][width];
    its column 0 is global column ``p_begin`` of a P-vector.  Returns float64
    [N][p_end-p_begin]."""
    lib = _load()
    elem, xptr, pitch, gptr, wptr, iptr, N, P, p_begin, p_end, keep = _common(
        x, grads, weights, idx, P, S, R, p_begin, p_end)
    out = np.empty((N, p_end - p_begin), dtype=np.float64)
    rc = lib.oracle_segment_aggregate(xptr, gptr, float(lr), elem, pitch, wptr, iptr, N, P, S, R,
                                      p_begin, p_end, out.ctypes.data)
    if rc != 0:
        raise ValueError("oracle_segment_aggregate: invalid arguments")
    return out


def segment_aggregate_ordered_f32(x, idx, S, R, weights=None, grads=None, lr=0.0, P=None,
                                  p_begin=0, p_end=None) -> np.ndarray:
    """The round in binary32, provider order self then peers ascending,
    weights normalised first, fused multiply-add accumulation.  Returns
    float32, or uint16 bf16 bit patterns for bf16 input."""
    lib = _load()
    elem, xptr, pitch, gptr, wptr, iptr, N, P, p_begin, p_end, keep = _common(
        x, grads, weights, idx, P, S, R, p_begin, p_end)
    out = np.empty((N, p_end - p_begin), dtype=np.float32 if elem == 4 else np.uint16)
    rc = lib.oracle_segment_aggregate_ordered_f32(xptr, gptr, float(lr), elem, pitch, wptr, iptr,
                                                  N, P, S, R, p_begin, p_end, out.ctypes.data)
    if rc != 0:
        raise ValueError("oracle_segment_aggregate_ordered_f32: invalid arguments")
    return out


def divergence(models, weights=None, mean_of=None) -> np.ndarray:
    """Eq. 7: rho_i = || models_i - weighted mean over the rows of mean_of || (binary64,
    Euclidean norm).  ``mean_of`` defaults to ``models``.  Arrays are float32 or uint16
    (bf16) [N][P]."""
    lib = _load()
    elem = 4 if models.dtype == np.float32 else 2
    mptr, P = _slab(models, elem)
    N = models.shape[0]
    sptr = None
    if mean_of is not None:
        sptr, P2 = _slab(mean_of, elem)
        if P2 != P or mean_of.shape[0] != N:
            raise ValueError("mean_of shape mismatch")
    wptr = None
    if weights is not None:
        weights = np.ascontiguousarray(weights, dtype=np.float32)
        wptr = weights.ctypes.data
    rho = np.zeros(N, dtype=np.float64)
    rc = lib.oracle_divergence(mptr, sptr, elem, wptr, N, P, rho.ctypes.data)
    if rc != 0:
        raise ValueError("oracle_divergence: invalid arguments")
    return rho


def select_peers_active(seed, rnd, N, S, R, active=None) -> np.ndarray:
    """Section 4.2: peers drawn from the ONLINE others only; rows of offline workers are -1."""
    lib = _load()
    idx = np.zeros((N, S, max(R, 0)), dtype=np.int32)
    aptr = None
    if active is not None:
        active = np.ascontiguousarray(active, dtype=np.uint8)
        aptr = active.ctypes.data
    rc = lib.oracle_select_peers_active(seed, rnd, N, S, R, aptr,
                                        idx.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)))
    if rc != 0:
        raise ValueError("oracle_select_peers_active: invalid arguments")
    return idx


def segment_aggregate_members(x, idx, S, R, weights=None, newcomer=None, ordered=False) -> np.ndarray:
    """Eq. 3 with Section 4.2's provider sets: self unless a newcomer, plus the
    non-negative idx entries.  binary64 result, or the fixed-order binary32 form."""
    lib = _load()
    elem = 4 if x.dtype == np.float32 else 2
    xptr, P = _slab(x, elem)
    N = x.shape[0]
    wptr = None
    if weights is not None:
        weights = np.ascontiguousarray(weights, dtype=np.float32)
        wptr = weights.ctypes.data
    nptr = None
    if newcomer is not None:
        newcomer = np.ascontiguousarray(newcomer, dtype=np.uint8)
        nptr = newcomer.ctypes.data
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    iptr = idx.ctypes.data if R > 0 else None
    if ordered:
        out = np.empty((N, P), dtype=np.float32 if elem == 4 else np.uint16)
    else:
        out = np.empty((N, P), dtype=np.float64)
    rc = lib.oracle_segment_aggregate_members(xptr, elem, wptr, iptr, nptr, N, P, S, R, 1 if ordered else 0,
                                              out.ctypes.data)
    if rc != 0:
        raise ValueError("oracle_segment_aggregate_members: invalid arguments")
    return out
