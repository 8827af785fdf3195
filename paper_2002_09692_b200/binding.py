"""ctypes binding of libsaps.so: the same names as the C ABI (include/saps.h) and nothing
but argument marshalling.  Every step of the gossip round runs in the CUDA library; there
is no Python or CPU fallback, and a missing library is an ImportError.

Pointer arguments accept a torch tensor, a numpy array, a ctypes array or a raw integer
address; streams accept a ``torch.cuda.Stream``, a raw handle, or None (torch's current
stream when torch is loaded, else the default stream).
"""
from __future__ import annotations

import ctypes
import os
import sys
from pathlib import Path

_LIB_PATH = Path(__file__).resolve().parent / "libsaps.so"

SAPS_OK = 0
SAPS_ERR_INVALID = -1
SAPS_ERR_PAIRS = -2
SAPS_ERR_CUDA = -3
SAPS_ERR_OVERFLOW = -4
SAPS_ERR_TIMEOUT = -5
SAPS_ERR_NOMEM = -6
SAPS_ERR_TOO_LARGE = -7
SAPS_NOALLOC_MAX_N = 134_217_728
SAPS_NEVER = -(1 << 62)
SAPS_SELECT_MAX_T = (1 << 62) - 1


def _load() -> ctypes.CDLL:
    if not _LIB_PATH.exists():
        raise ImportError(
            f"{_LIB_PATH} is missing: build it with `python -m paper_2002_09692_b200.build` "
            "(there is no fallback path)")
    return ctypes.CDLL(str(_LIB_PATH))


_lib = _load()

_vp, _u64, _u32, _i32 = ctypes.c_void_p, ctypes.c_uint64, ctypes.c_uint32, ctypes.c_int
_f32, _f64 = ctypes.c_float, ctypes.c_double

_SIGNATURES = {
    "saps_create": (_i32, [_i32, _u64, _u64, ctypes.POINTER(_vp)]),
    "saps_create_ld": (_i32, [_i32, _u64, _u64, _u64, ctypes.POINTER(_vp)]),
    "saps_set_column_offset": (_i32, [_vp, _u64]),
    "saps_destroy": (_i32, [_vp]),
    "saps_round_key": (None, [_u64, _u64, ctypes.POINTER(_u32), ctypes.POINTER(_u32)]),
    "saps_threshold": (_u64, [_f64]),
    "saps_mask": (_i32, [_vp, _u64, _f64, _vp, _vp]),
    "saps_round": (_i32, [_vp, _vp, _vp, _f32, _vp, _u64, _f64, _vp]),
    "saps_round_pack": (_i32, [_vp, _vp, _vp, _f32, _vp, _u64, _f64, _vp, _vp, _vp, _vp]),
    "saps_round_pack_rows": (_i32, [_vp, _vp, _vp, _f32, _vp, _u64, _f64, _vp, _vp, _vp, _vp]),
    "saps_pack_capacity": (_u64, [_vp, _f64]),
    "saps_set_pack_capacity": (_i32, [_vp, _u64]),
    "saps_pack": (_i32, [_vp, _vp, _u64, _f64, _vp, _vp, _vp, _vp]),
    "saps_pack_noalloc": (_i32, [_vp, _vp, _u64, _f64, _vp, _vp, _vp, _vp, _vp]),
    "saps_set_select_params": (_i32, [_vp, _f64, _i32]),
    "saps_select_peers": (_i32, [_vp, _vp, _u64, _vp]),
    "saps_select_reset": (_i32, [_vp]),
    "saps_get_select_state": (_i32, [_vp, _vp, ctypes.POINTER(_u64)]),
    "saps_set_select_state": (_i32, [_vp, _vp, _u64]),
    "saps_run_rounds": (_i32, [_vp, _vp, _vp, _f32, _u64, _u64, _f64, _vp, _vp, _vp, _vp, _vp]),
    "saps_run_rounds_pack": (_i32, [_vp, _vp, _vp, _f32, _u64, _u64, _f64, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp]),
    "saps_set_update_order": (_i32, [_vp, _i32]),
    "saps_set_staging": (_i32, [_vp, _i32]),
    "saps_set_run_ahead": (_i32, [_vp, _i32]),
    "saps_unpack_avg": (_i32, [_vp, _vp, _vp, _vp, _vp, _f64, _vp, _vp]),
    "saps_unpack_avg_rows": (_i32, [_vp, _vp, _vp, _vp, _vp, _f64, _vp, _vp]),
    "saps_consensus_distance": (_i32, [_vp, _vp, _vp, _vp]),
    "saps_comm_stats": (_i32, [_vp, _vp, _vp, _u64, _f64, _vp]),
    "saps_debug_inject": (_i32, [_vp, _u32, _u32]),
    "saps_debug_staging_wait": (_i32, [_vp, _i32]),
    "saps_round_host": (_i32, [_vp, _vp, _vp, _f32, _vp, _u64, _f64, _vp, _vp]),
    "saps_round_pack_host": (_i32, [_vp, _vp, _vp, _f32, _vp, _u64, _f64, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp]),
    "saps_set_host_pipeline": (_i32, [_vp, _u64, _i32]),
    "saps_set_timing_events": (_i32, [_vp, _vp, _vp]),
    "saps_status": (_i32, [_vp, _vp, ctypes.POINTER(_i32)]),
    "saps_strerror": (ctypes.c_char_p, [_i32]),
}
for _name, (_res, _args) in _SIGNATURES.items():
    _fn = getattr(_lib, _name)
    _fn.restype = _res
    _fn.argtypes = _args

EXPORTS = tuple(_SIGNATURES)


class SapsError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {saps_strerror(status)} ({status})")


def _check(status: int, where: str) -> None:
    if status != SAPS_OK:
        raise SapsError(status, where)


def _ptr(a):
    """Address of a buffer-like argument (None -> NULL)."""
    if a is None:
        return None
    if isinstance(a, int):
        return a
    if hasattr(a, "data_ptr"):          # torch tensor
        return a.data_ptr()
    if hasattr(a, "ctypes"):            # numpy array
        return a.ctypes.data
    return ctypes.cast(a, ctypes.c_void_p).value


def _stream(s):
    if s is None:
        torch = sys.modules.get("torch")
        if torch is not None and torch.cuda.is_available():
            return torch.cuda.current_stream().cuda_stream
        return None
    if isinstance(s, int):
        return s
    return s.cuda_stream


def _pairs(pairs, n=None):
    seq = [int(v) for v in pairs]
    return (ctypes.c_int32 * len(seq))(*seq)


# ---- the C ABI, one Python function per export ---------------------------------------------

def saps_create(n: int, N: int, seed: int):
    h = _vp()
    _check(_lib.saps_create(n, N, seed, ctypes.byref(h)), "saps_create")
    return h


def saps_create_ld(n: int, N: int, ld: int, seed: int):
    h = _vp()
    _check(_lib.saps_create_ld(n, N, ld, seed, ctypes.byref(h)), "saps_create_ld")
    return h


def saps_set_column_offset(ctx, col_offset: int) -> None:
    _check(_lib.saps_set_column_offset(ctx, col_offset), "saps_set_column_offset")


def saps_destroy(ctx) -> None:
    _check(_lib.saps_destroy(ctx), "saps_destroy")


def saps_round_key(seed: int, t: int):
    k0, k1 = _u32(), _u32()
    _lib.saps_round_key(seed, t, ctypes.byref(k0), ctypes.byref(k1))
    return k0.value, k1.value


def saps_threshold(keep_frac: float) -> int:
    return int(_lib.saps_threshold(keep_frac))


def saps_mask(ctx, t, keep_frac, out_bits, stream=None) -> None:
    _check(_lib.saps_mask(ctx, t, keep_frac, _ptr(out_bits), _stream(stream)), "saps_mask")


def saps_round(ctx, x, g, lr, pairs, t, keep_frac, stream=None) -> None:
    _check(_lib.saps_round(ctx, _ptr(x), _ptr(g), lr, _pairs(pairs), t, keep_frac, _stream(stream)),
           "saps_round")


def saps_round_pack(ctx, x, g, lr, pairs, t, keep_frac, out_vals, out_idx, out_count, stream=None) -> None:
    _check(_lib.saps_round_pack(ctx, _ptr(x), _ptr(g), lr, _pairs(pairs), t, keep_frac, _ptr(out_vals),
                                _ptr(out_idx), _ptr(out_count), _stream(stream)), "saps_round_pack")


def saps_round_pack_rows(ctx, x, g, lr, pairs, t, keep_frac, out_rows, out_idx, out_count, stream=None) -> None:
    """out_rows: device array of n 64-bit addresses (e.g. an int64 tensor), one destination per worker."""
    _check(_lib.saps_round_pack_rows(ctx, _ptr(x), _ptr(g), lr, _pairs(pairs), t, keep_frac, _ptr(out_rows),
                                     _ptr(out_idx), _ptr(out_count), _stream(stream)), "saps_round_pack_rows")


def saps_pack_capacity(ctx, keep_frac: float) -> int:
    return int(_lib.saps_pack_capacity(ctx, keep_frac))


def saps_set_pack_capacity(ctx, cap: int) -> None:
    _check(_lib.saps_set_pack_capacity(ctx, cap), "saps_set_pack_capacity")


def saps_pack(ctx, x, t, keep_frac, out_vals, out_idx, out_count, stream=None) -> None:
    _check(_lib.saps_pack(ctx, _ptr(x), t, keep_frac, _ptr(out_vals), _ptr(out_idx), _ptr(out_count),
                          _stream(stream)), "saps_pack")


def saps_pack_noalloc(ctx, x, t, keep_frac, out_vals, out_idx, out_count, out_status=None, stream=None) -> None:
    """saps_pack on the library's built-in scratch array: for callers that may not allocate
    device memory.  Calls share that array, so keep them on one stream (or order them)."""
    _check(_lib.saps_pack_noalloc(ctx, _ptr(x), t, keep_frac, _ptr(out_vals), _ptr(out_idx), _ptr(out_count),
                                  _ptr(out_status), _stream(stream)), "saps_pack_noalloc")


def saps_set_select_params(ctx, b_thres: float, t_thres: int) -> None:
    _check(_lib.saps_set_select_params(ctx, b_thres, t_thres), "saps_set_select_params")


def saps_select_peers(ctx, bandwidth, t: int, n: int):
    """bandwidth: n x n row-major float64 (numpy array or flat sequence). Returns the pairs list."""
    if hasattr(bandwidth, "ctypes"):
        import numpy as np
        b = np.ascontiguousarray(bandwidth, dtype=np.float64)
        if b.size != n * n:
            raise ValueError("bandwidth must be n x n")
        bp = b.ctypes.data
    else:
        flat = [float(v) for v in bandwidth]
        if len(flat) != n * n:
            raise ValueError("bandwidth must be n x n")
        b = (ctypes.c_double * (n * n))(*flat)
        bp = ctypes.addressof(b)
    out = (ctypes.c_int32 * n)()
    _check(_lib.saps_select_peers(ctx, bp, t, out), "saps_select_peers")
    return list(out)


def saps_select_reset(ctx) -> None:
    _check(_lib.saps_select_reset(ctx), "saps_select_reset")


def saps_get_select_state(ctx, n: int):
    R = (ctypes.c_int64 * (n * n))()
    last = _u64()
    _check(_lib.saps_get_select_state(ctx, R, ctypes.byref(last)), "saps_get_select_state")
    return [list(R[i * n:(i + 1) * n]) for i in range(n)], last.value


def saps_set_select_state(ctx, R, last_t: int) -> None:
    flat = [int(v) for row in R for v in row]
    arr = (ctypes.c_int64 * len(flat))(*flat)
    _check(_lib.saps_set_select_state(ctx, arr, last_t), "saps_set_select_state")


def saps_run_rounds(ctx, x, g, lr, t_first, T, keep_frac, pairs_list=None, bandwidth=None,
                    out_pairs_log=None, stream=None, lr_list=None) -> None:
    """pairs_list: T x n int32 numpy array or None; bandwidth: n x n float64 numpy array or
    None; out_pairs_log: T x n int32 numpy array to fill, or None; lr_list: T float32 numpy
    array (a learning rate per round) or None."""
    _check(_lib.saps_run_rounds(ctx, _ptr(x), _ptr(g), lr, t_first, T, keep_frac, _ptr(lr_list),
                                _ptr(pairs_list), _ptr(bandwidth), _ptr(out_pairs_log), _stream(stream)),
           "saps_run_rounds")


def saps_run_rounds_pack(ctx, x, g, lr, t_first, T, keep_frac, out_vals, out_idx, out_counts, pairs_list=None,
                         bandwidth=None, out_pairs_log=None, stream=None, lr_list=None) -> None:
    _check(_lib.saps_run_rounds_pack(ctx, _ptr(x), _ptr(g), lr, t_first, T, keep_frac, _ptr(lr_list),
                                     _ptr(pairs_list), _ptr(bandwidth), _ptr(out_pairs_log), _ptr(out_vals),
                                     _ptr(out_idx), _ptr(out_counts), _stream(stream)), "saps_run_rounds_pack")


SAPS_ORDER_SGD_FIRST = 0
SAPS_ORDER_GOSSIP_FIRST = 1


def saps_set_update_order(ctx, order: int) -> None:
    _check(_lib.saps_set_update_order(ctx, order), "saps_set_update_order")


SAPS_STAGING_AUTO, SAPS_STAGING_REGISTERS, SAPS_STAGING_BULK = 0, 1, 2


def saps_set_staging(ctx, staging: int) -> None:
    _check(_lib.saps_set_staging(ctx, staging), "saps_set_staging")


def saps_set_run_ahead(ctx, enabled: bool) -> None:
    _check(_lib.saps_set_run_ahead(ctx, int(bool(enabled))), "saps_set_run_ahead")


def saps_unpack_avg(ctx, x, recv_vals, idx, count, keep_frac, pairs=None, stream=None) -> None:
    _check(_lib.saps_unpack_avg(ctx, _ptr(x), _ptr(recv_vals), _ptr(idx), _ptr(count), keep_frac,
                                None if pairs is None else _pairs(pairs), _stream(stream)), "saps_unpack_avg")


def saps_unpack_avg_rows(ctx, x, recv_vals, idx, count, keep_frac, src_rows, stream=None) -> None:
    _check(_lib.saps_unpack_avg_rows(ctx, _ptr(x), _ptr(recv_vals), _ptr(idx), _ptr(count), keep_frac,
                                     _pairs(src_rows), _stream(stream)), "saps_unpack_avg_rows")


def saps_consensus_distance(ctx, x, out, stream=None) -> None:
    _check(_lib.saps_consensus_distance(ctx, _ptr(x), _ptr(out), _stream(stream)), "saps_consensus_distance")


def saps_comm_stats(ctx, bandwidth, pairs, count: int, bits_per_s_per_unit: float = 1e6):
    """bandwidth: n x n float64 numpy array.  Returns a dict of the five figures."""
    out = (ctypes.c_double * 5)()
    _check(_lib.saps_comm_stats(ctx, _ptr(bandwidth), _pairs(pairs), count, bits_per_s_per_unit, out),
           "saps_comm_stats")
    keys = ("values_per_worker", "bytes_per_worker", "bottleneck_bandwidth", "mean_bandwidth", "comm_time_s")
    return dict(zip(keys, out))


def saps_debug_inject(ctx, skip_tile: int, spin_limit: int) -> None:
    _check(_lib.saps_debug_inject(ctx, skip_tile, spin_limit), "saps_debug_inject")


def saps_debug_staging_wait(ctx, give_up: bool) -> None:
    _check(_lib.saps_debug_staging_wait(ctx, 1 if give_up else 0), "saps_debug_staging_wait")


def saps_round_host(ctx, x_host, g_host, lr, pairs, t, keep_frac, d_x, d_g) -> None:
    _check(_lib.saps_round_host(ctx, _ptr(x_host), _ptr(g_host), lr, _pairs(pairs), t, keep_frac,
                                _ptr(d_x), _ptr(d_g)), "saps_round_host")


def saps_round_pack_host(ctx, x_host, g_host, lr, pairs, t, keep_frac, d_x, d_g, out_vals_host,
                         out_idx_host, out_count_host, d_vals, d_idx, d_count) -> None:
    _check(_lib.saps_round_pack_host(ctx, _ptr(x_host), _ptr(g_host), lr, _pairs(pairs), t, keep_frac,
                                     _ptr(d_x), _ptr(d_g), _ptr(out_vals_host), _ptr(out_idx_host),
                                     _ptr(out_count_host), _ptr(d_vals), _ptr(d_idx), _ptr(d_count)),
           "saps_round_pack_host")


def saps_set_host_pipeline(ctx, chunk_columns: int = 0, lanes: int = 0) -> None:
    _check(_lib.saps_set_host_pipeline(ctx, chunk_columns, lanes), "saps_set_host_pipeline")


def saps_set_timing_events(ctx, before, after) -> None:
    """before/after: torch.cuda.Event (already recorded once or created with enable_timing) or
    raw cudaEvent_t handles, or None to switch the hook off."""
    def handle(e):
        if e is None or isinstance(e, int):
            return e
        return e.cuda_event
    _check(_lib.saps_set_timing_events(ctx, handle(before), handle(after)), "saps_set_timing_events")


def saps_status(ctx, stream=None) -> int:
    st = _i32()
    _check(_lib.saps_status(ctx, _stream(stream), ctypes.byref(st)), "saps_status")
    return st.value


def saps_strerror(status: int) -> str:
    return _lib.saps_strerror(status).decode()
