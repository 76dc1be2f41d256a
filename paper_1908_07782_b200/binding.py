"""ctypes binding of libcombo_b200.so: same names as the C ABI, argument
marshalling only.  Tensors are torch tensors (device memory and streams come
from PyTorch); every step of the round runs inside the library's kernels.
There is no fallback: a missing library raises."""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libcombo_b200.so")
_lib = None

COMBO_OK = 0
PATH_AUTO, PATH_DIRECT, PATH_STAGED, PATH_TILE, PATH_DIRECT_NAIVE = 0, 1, 2, 5, 6


class ComboError(RuntimeError):
    def __init__(self, status: int, where: str):
        lib = load()
        msg = lib.combo_status_string(status).decode()
        detail = lib.combo_last_cuda_error().decode()
        super().__init__("%s: %s%s" % (where, msg, (" (%s)" % detail) if status == 4 and detail else ""))
        self.status = status


def load():
    """Loads the shared library; raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(
            "libcombo_b200.so is missing (%s); build it with "
            "`python -m paper_1908_07782_b200.build` -- there is no fallback path" % LIB_PATH)
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, i64, u32, u64, f32 = (ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_uint32,
                                   ctypes.c_uint64, ctypes.c_float)
    sigs = {
        "combo_select_peers": [u64, u32, i32, i32, i32, vp],
        "combo_select_peers_async": [u64, u32, i32, i32, i32, vp, vp],
        "combo_segment_aggregate": [vp, vp, vp, vp, i32, i64, i32, i32, vp],
        "combo_segment_aggregate_bf16": [vp, vp, vp, vp, i32, i64, i32, i32, vp],
        "combo_segment_aggregate_sgd": [vp, vp, f32, vp, vp, vp, i32, i64, i32, i32, vp],
        "combo_segment_aggregate_cols": [vp, vp, f32, vp, i32, vp, vp, i32, i64, i32, i32, i64, i64,
                                         i64, vp],
        "combo_validate_idx": [vp, i32, i32, i32, vp, vp],
        "combo_segment_aggregate_rows": [vp, vp, i64, i32, vp, vp, i32, i64, i32, i32, i32, i32, vp],
        "combo_check_rows": [vp, i32, vp, vp],
        "combo_select_peers_online": [u64, u32, i32, i32, i32, vp, vp, vp],
        "combo_segment_aggregate_members": [vp, vp, i32, vp, vp, vp, i32, i64, i32, i32, vp],
        "combo_round_host": [vp, vp, f32, vp, i32, vp, u64, u32, i32, i32, i64, i32, i32, vp, vp, vp,
                             vp, vp, vp, vp],
        "combo_aggregation_divergence": [vp, vp, i32, vp, i32, i64, vp, vp, ctypes.c_size_t, vp],
        "combo_aggregation_divergence_noalloc": [vp, vp, i32, vp, i32, i64, vp, vp],
        "combo_debug_dead_wait": [vp],
        "combo_device_status": [],
        "combo_last_kernel_path": [],
        "combo_version": [],
    }
    for name, args in sigs.items():
        fn = getattr(lib, name)
        fn.argtypes = args
        fn.restype = ctypes.c_int
    lib.combo_divergence_scratch_bytes.argtypes = [i32]
    lib.combo_divergence_scratch_bytes.restype = ctypes.c_size_t
    lib.combo_set_kernel_path.argtypes = [i32]
    lib.combo_set_kernel_path.restype = None
    lib.combo_set_tuning.argtypes = [i32, i32]
    lib.combo_set_tuning.restype = None
    lib.combo_max_launch_columns.argtypes = []
    lib.combo_max_launch_columns.restype = ctypes.c_int64
    lib.combo_set_launch_columns.argtypes = [i64]
    lib.combo_set_launch_columns.restype = None
    lib.combo_set_launch_overlap.argtypes = [i32]
    lib.combo_set_launch_overlap.restype = None
    lib.combo_status_string.argtypes = [i32]
    lib.combo_status_string.restype = ctypes.c_char_p
    lib.combo_last_cuda_error.argtypes = []
    lib.combo_last_cuda_error.restype = ctypes.c_char_p
    _lib = lib
    return lib


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _check(status: int, where: str):
    if status != COMBO_OK:
        raise ComboError(status, where)


def combo_select_peers(seed: int, rnd: int, N: int, S: int, R: int, idx_out: torch.Tensor,
                       stream=None) -> torch.Tensor:
    """Peer table for (seed, round) into idx_out (int32 [N][S][R], device), on
    the current torch stream (or ``stream``)."""
    _check(load().combo_select_peers_async(seed, rnd, N, S, R, _ptr(idx_out), _stream(stream)),
           "combo_select_peers")
    return idx_out


def combo_select_peers_default_stream(seed, rnd, N, S, R, idx_out):
    """The stream-less C entry point (legacy default stream)."""
    _check(load().combo_select_peers(seed, rnd, N, S, R, _ptr(idx_out)), "combo_select_peers")
    return idx_out


def combo_segment_aggregate(params_in, params_out, weights, idx, N, P, S, R, stream=None):
    _check(load().combo_segment_aggregate(_ptr(params_in), _ptr(params_out), _ptr(weights), _ptr(idx),
                                          N, P, S, R, _stream(stream)), "combo_segment_aggregate")
    return params_out


def combo_segment_aggregate_bf16(params_in, params_out, weights, idx, N, P, S, R, stream=None):
    _check(load().combo_segment_aggregate_bf16(_ptr(params_in), _ptr(params_out), _ptr(weights),
                                               _ptr(idx), N, P, S, R, _stream(stream)),
           "combo_segment_aggregate_bf16")
    return params_out


def combo_segment_aggregate_sgd(params_in, grads, lr, params_out, weights, idx, N, P, S, R,
                                stream=None):
    _check(load().combo_segment_aggregate_sgd(_ptr(params_in), _ptr(grads), lr, _ptr(params_out),
                                              _ptr(weights), _ptr(idx), N, P, S, R, _stream(stream)),
           "combo_segment_aggregate_sgd")
    return params_out


def combo_segment_aggregate_cols(params_in, grads, lr, params_out, elem_bytes, weights, idx, N,
                                 P_total, S, R, p_begin, width, pitch, stream=None):
    _check(load().combo_segment_aggregate_cols(_ptr(params_in), _ptr(grads), lr, _ptr(params_out),
                                               elem_bytes, _ptr(weights), _ptr(idx), N, P_total, S, R,
                                               p_begin, width, pitch, _stream(stream)),
           "combo_segment_aggregate_cols")
    return params_out


def _host_bytes(flags, N):
    """N flag bytes in host memory for the C side (None stays NULL)."""
    if flags is None:
        return None, None
    buf = (ctypes.c_uint8 * N)(*[1 if bool(f) else 0 for f in flags])
    return buf, ctypes.cast(buf, ctypes.c_void_p)


def combo_segment_aggregate_rows(rows, out, out_pitch, elem_bytes, weights, idx, N, P, S, R, w_begin, n_local,
                                 stream=None):
    """Worker-sharded Eq. 3: ``rows`` is a device int64 tensor of N row addresses (local or
    peer memory), ``out`` holds the n_local hosted workers' new models, [n_local][out_pitch]."""
    _check(load().combo_segment_aggregate_rows(_ptr(rows), _ptr(out), out_pitch, elem_bytes, _ptr(weights),
                                               _ptr(idx), N, P, S, R, w_begin, n_local, _stream(stream)),
           "combo_segment_aggregate_rows")
    return out


def combo_check_rows(rows, N, stream=None) -> int:
    """0 when all N row addresses are non-null and 16-byte aligned, else 1 + the first bad row."""
    flag = torch.zeros(1, dtype=torch.int32, device=rows.device)
    _check(load().combo_check_rows(_ptr(rows), N, _stream(stream), _ptr(flag)), "combo_check_rows")
    return int(flag.item())


def combo_select_peers_online(seed, rnd, N, S, R, online, idx_out, stream=None):
    """Section 4.2: peers drawn from the online others only; ``online`` is a host
    sequence of N flags (None = all online).  Offline workers' rows become -1."""
    keep, ptr = _host_bytes(online, N)
    _check(load().combo_select_peers_online(seed, rnd, N, S, R, ptr, _ptr(idx_out), _stream(stream)),
           "combo_select_peers_online")
    return idx_out


def combo_segment_aggregate_members(params_in, params_out, weights, idx, newcomer, N, P, S, R, stream=None):
    """Eq. 3 where newcomers (host sequence of N flags, or None) aggregate without their
    own model and negative idx entries are skipped."""
    keep, ptr = _host_bytes(newcomer, N)
    _check(load().combo_segment_aggregate_members(_ptr(params_in), _ptr(params_out), params_in.element_size(),
                                                  _ptr(weights), _ptr(idx), ptr, N, P, S, R, _stream(stream)),
           "combo_segment_aggregate_members")
    return params_out


def combo_validate_idx(idx, N, S, R, dev_flag, stream=None):
    _check(load().combo_validate_idx(_ptr(idx), N, S, R, _stream(stream), _ptr(dev_flag)),
           "combo_validate_idx")
    return dev_flag


def combo_round_host(h_params_in, h_grads, lr, h_params_out, elem_bytes, h_weights, seed, rnd, rounds,
                     N, P, S, R, d_in, d_grads, d_out, d_weights, d_idx, h_idx_out=None, stream=None):
    """``rounds`` chained rounds from host tensors (pinned for speed) through
    caller-owned device buffers; returns after the result is in h_params_out."""
    _check(load().combo_round_host(_ptr(h_params_in), _ptr(h_grads), lr, _ptr(h_params_out),
                                   elem_bytes, _ptr(h_weights), seed, rnd, rounds, N, P, S, R, _ptr(d_in),
                                   _ptr(d_grads), _ptr(d_out), _ptr(d_weights), _ptr(d_idx),
                                   _ptr(h_idx_out), _stream(stream)), "combo_round_host")
    return h_params_out


def combo_divergence_scratch_bytes(N: int) -> int:
    return int(load().combo_divergence_scratch_bytes(N))


def combo_aggregation_divergence(models, mean_of, elem_bytes, weights, N, P, rho_out, scratch, stream=None):
    """Eq. 7 for all workers: rho_out (float64 [N], device) = distance of each row of
    ``models`` from the weighted mean over the rows of ``mean_of`` (or of ``models``).
    ``scratch`` is a device tensor of at least combo_divergence_scratch_bytes(N) bytes."""
    _check(load().combo_aggregation_divergence(_ptr(models), _ptr(mean_of), elem_bytes, _ptr(weights), N, P,
                                               _ptr(rho_out), _ptr(scratch),
                                               scratch.numel() * scratch.element_size(), _stream(stream)),
           "combo_aggregation_divergence")
    return rho_out


def combo_aggregation_divergence_noalloc(models, mean_of, elem_bytes, weights, N, P, rho_out, stream=None):
    """The same measurement for callers that cannot allocate device memory: the
    partial sums go to a fixed 1 MiB array inside the library instead of a
    caller-supplied scratch tensor.  At most 128 workers; all calls on a device
    share that array, so issue them on one stream."""
    _check(load().combo_aggregation_divergence_noalloc(_ptr(models), _ptr(mean_of), elem_bytes, _ptr(weights), N,
                                                       P, _ptr(rho_out), _stream(stream)),
           "combo_aggregation_divergence_noalloc")
    return rho_out


def combo_device_status():
    _check(load().combo_device_status(), "combo_device_status")


def combo_last_kernel_path() -> int:
    return load().combo_last_kernel_path()


def combo_set_kernel_path(path: int) -> None:
    load().combo_set_kernel_path(path)


def combo_set_tuning(tile_elems: int = 0, stages: int = 0) -> None:
    load().combo_set_tuning(tile_elems, stages)


def combo_set_launch_overlap(on: bool = True) -> None:
    load().combo_set_launch_overlap(1 if on else 0)


def combo_max_launch_columns() -> int:
    return int(load().combo_max_launch_columns())


def combo_set_launch_columns(columns: int = 0) -> None:
    load().combo_set_launch_columns(columns)


def combo_debug_dead_wait(stream=None) -> None:
    """Enqueues the self-check kernel whose bounded wait runs out (see the header)."""
    _check(load().combo_debug_dead_wait(_stream(stream)), "combo_debug_dead_wait")


def combo_version() -> int:
    return load().combo_version()
