"""CPU oracle for the SAPS-PSGD gossip round and peer selection.

TEST INFRASTRUCTURE ONLY.  The test-suite, the smoke check and the benchmark's
CPU-baseline leg are the only callers; the product path never imports this
package, and this package never imports the product.

``round`` side: ``saps_oracle.c`` (plain C, one thread, fp32 with every
operation rounded separately), reached through ctypes.
``peer selection`` side: ``peer_selection.py`` (plain Python, Algorithm 3).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "saps_oracle.c"
_LIB = _HERE / "libsaps_oracle.so"

# -ffp-contract=off: no fused multiply-add, so each fp32 operation rounds once.
_CFLAGS = ["-O2", "-std=c11", "-fPIC", "-shared", "-ffp-contract=off", "-fno-fast-math"]


def build(force: bool = False) -> Path:
    """Compile the C oracle with gcc if the shared object is missing or stale."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".tmp{os.getpid()}.so")
        subprocess.run(["gcc", *_CFLAGS, "-o", str(tmp), str(_SRC), "-lm"], check=True)
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _bind(lib):
    """Declare the C signatures on a loaded oracle library."""
    u32, u64, i32 = ctypes.c_uint32, ctypes.c_uint64, ctypes.c_int
    vp, dbl, f32 = ctypes.c_void_p, ctypes.c_double, ctypes.c_float
    lib.orc_mix.restype = u32
    lib.orc_mix.argtypes = [u32]
    lib.orc_round_key.restype = None
    lib.orc_round_key.argtypes = [u64, u64, ctypes.POINTER(u32), ctypes.POINTER(u32)]
    lib.orc_hash.restype = u32
    lib.orc_hash.argtypes = [u32, u32, u32]
    lib.orc_threshold.restype = u64
    lib.orc_threshold.argtypes = [dbl]
    lib.orc_mask.restype = None
    lib.orc_mask.argtypes = [u64, u64, dbl, u64, vp]
    lib.orc_sgd.restype = None
    lib.orc_sgd.argtypes = [i32, u64, vp, vp, f32]
    lib.orc_pack.restype = u64
    lib.orc_pack.argtypes = [i32, u64, vp, vp, u64, vp, vp]
    lib.orc_pair_average.restype = None
    lib.orc_pair_average.argtypes = [i32, u64, vp, vp, vp]
    lib.orc_round.restype = None
    lib.orc_round.argtypes = [i32, u64, vp, vp, f32, vp, u64, u64, dbl, vp]
    lib.orc_round_eq7.restype = None
    lib.orc_round_eq7.argtypes = [i32, u64, vp, vp, f32, vp, u64, u64, dbl, vp]
    lib.orc_unpack_avg.restype = None
    lib.orc_unpack_avg.argtypes = [i32, u64, vp, vp, u64, vp, u64]
    lib.orc_consensus_distance.restype = dbl
    lib.orc_consensus_distance.argtypes = [i32, u64, vp]
    return lib


def _c():
    global _lib
    if _lib is None:
        _lib = _bind(ctypes.CDLL(str(build())))
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _f32_matrix(a, name, writable=False):
    if not (isinstance(a, np.ndarray) and a.dtype == np.float32 and a.ndim == 2
            and a.flags.c_contiguous):
        raise TypeError(f"{name} must be a C-contiguous float32 [n, N] array")
    if writable and not a.flags.writeable:
        raise TypeError(f"{name} must be writable")
    return a


def mix(v: int) -> int:
    return int(_c().orc_mix(v & 0xFFFFFFFF))


def round_key(seed: int, t: int) -> tuple[int, int]:
    k0, k1 = ctypes.c_uint32(), ctypes.c_uint32()
    _c().orc_round_key(seed, t, ctypes.byref(k0), ctypes.byref(k1))
    return int(k0.value), int(k1.value)


def hash_k(k: int, k0: int, k1: int) -> int:
    return int(_c().orc_hash(k & 0xFFFFFFFF, k0, k1))


def threshold(keep_frac: float) -> int:
    return int(_c().orc_threshold(float(keep_frac)))


def mask(seed: int, t: int, keep_frac: float, N: int) -> np.ndarray:
    """The round-t mask as a uint8 vector of N zeros and ones."""
    m = np.empty(N, dtype=np.uint8)
    _c().orc_mask(seed, t, float(keep_frac), N, _ptr(m))
    return m


def sgd(x: np.ndarray, g, lr: float) -> None:
    """In place ``x -= lr*g`` (two roundings per element); ``g=None`` is a no-op."""
    _f32_matrix(x, "x", True)
    if g is not None:
        _f32_matrix(g, "g")
        assert g.shape == x.shape
    _c().orc_sgd(x.shape[0], x.shape[1], _ptr(x), _ptr(g), float(lr))


def pack(a: np.ndarray, m: np.ndarray, cap: int | None = None):
    """Return ``(vals[n, cap], idx[cap], count)`` for the kept columns of ``a``.

    Slots at and beyond ``count`` are left at zero; ``count`` may exceed ``cap``.
    """
    _f32_matrix(a, "a")
    n, N = a.shape
    assert m.dtype == np.uint8 and m.shape == (N,)
    if cap is None:
        cap = int(m.sum())
    vals = np.zeros((n, cap), dtype=np.float32)
    idx = np.zeros(cap, dtype=np.uint32)
    count = int(_c().orc_pack(n, N, _ptr(a), _ptr(m), cap, _ptr(vals), _ptr(idx)))
    return vals, idx, count


def pair_average(a: np.ndarray, pairs, m: np.ndarray) -> None:
    _f32_matrix(a, "a", True)
    n, N = a.shape
    p = np.ascontiguousarray(pairs, dtype=np.int32)
    _check_pairs(p, n)
    assert m.dtype == np.uint8 and m.shape == (N,)
    _c().orc_pair_average(n, N, _ptr(a), _ptr(p), _ptr(m))


def gossip_round(x: np.ndarray, g, lr: float, pairs, seed: int, t: int,
                 keep_frac: float) -> np.ndarray:
    """One whole round in place on ``x``; returns the round's mask."""
    _f32_matrix(x, "x", True)
    n, N = x.shape
    if g is not None:
        _f32_matrix(g, "g")
        assert g.shape == x.shape
    p = np.ascontiguousarray(pairs, dtype=np.int32)
    _check_pairs(p, n)
    m = np.empty(N, dtype=np.uint8)
    _c().orc_round(n, N, _ptr(x), _ptr(g), float(lr), _ptr(p), seed, t, float(keep_frac),
                   _ptr(m))
    return m


def gossip_round_eq7(x: np.ndarray, g, lr: float, pairs, seed: int, t: int,
                     keep_frac: float) -> np.ndarray:
    """One round in the order of Eq. 7 (average the current models, then subtract the
    gradient step), in place on ``x``; returns the round's mask."""
    _f32_matrix(x, "x", True)
    n, N = x.shape
    if g is not None:
        _f32_matrix(g, "g")
        assert g.shape == x.shape
    p = np.ascontiguousarray(pairs, dtype=np.int32)
    _check_pairs(p, n)
    m = np.empty(N, dtype=np.uint8)
    _c().orc_round_eq7(n, N, _ptr(x), _ptr(g), float(lr), _ptr(p), seed, t, float(keep_frac),
                       _ptr(m))
    return m


def unpack_avg(x: np.ndarray, recv: np.ndarray, idx: np.ndarray, count: int) -> None:
    """In place: x[i, idx[r]] = (x[i, idx[r]] + recv[i, r]) / 2 for r < count."""
    _f32_matrix(x, "x", True)
    _f32_matrix(recv, "recv")
    assert recv.shape[0] == x.shape[0] and idx.dtype == np.uint32 and idx.flags.c_contiguous
    assert count <= idx.shape[0]
    _c().orc_unpack_avg(x.shape[0], x.shape[1], _ptr(x), _ptr(recv), recv.shape[1], _ptr(idx),
                        int(count))


def consensus_distance(x: np.ndarray) -> float:
    """|| X - mean over workers ||_F^2 in double precision."""
    _f32_matrix(x, "x")
    return float(_c().orc_consensus_distance(x.shape[0], x.shape[1], _ptr(x)))


def _check_pairs(p: np.ndarray, n: int) -> None:
    if p.shape != (n,):
        raise ValueError("pairs must have n entries")
    for i in range(n):
        j = int(p[i])
        if not (0 <= j < n) or int(p[j]) != i:
            raise ValueError("pairs is not an involution")
