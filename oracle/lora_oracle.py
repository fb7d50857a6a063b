"""ctypes front end of the CPU oracle (oracle/lora_oracle.c).

TEST INFRASTRUCTURE.  Only tests, the smoke check and the benchmark's CPU
baseline may import this module.  It imports nothing from the CUDA package.

The oracle evaluates, in fp64 and as the plain definition,
``y = y_base + s_i * (x . A_i) . B_i`` per token (paper Section 2.2 describes
the two low-rank matrices whose activations are added to the backbone layer
output; Section 1 says they stay unmerged over a shared backbone), and the
stable group-by-slot segment metadata.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading
from typing import Dict, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "lora_oracle.c")
_LIB = os.path.join(_HERE, "liblora_oracle.so")
_lock = threading.Lock()
_lib = None

_c_i32p = ctypes.POINTER(ctypes.c_int32)
_c_f64p = ctypes.POINTER(ctypes.c_double)


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP over tokens only)."""
    with _lock:
        if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
            tmp = _LIB + ".tmp.%d" % os.getpid()
            subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11",
                                   "-o", tmp, _SRC])
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.lora_oracle_apply.restype = ctypes.c_int64
        lib.lora_oracle_apply.argtypes = [
            ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32,
            _c_f64p, ctypes.c_int64, _c_f64p, ctypes.c_int64, _c_i32p,
            ctypes.POINTER(_c_f64p), ctypes.POINTER(_c_f64p),
            _c_i32p, _c_f64p, _c_i32p, _c_f64p, ctypes.c_int64, ctypes.c_int32]
        lib.lora_oracle_build_segments.restype = ctypes.c_int32
        lib.lora_oracle_build_segments.argtypes = (
            [ctypes.c_int32, ctypes.c_int32, _c_i32p, _c_i32p, _c_i32p,
             ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32] + [_c_i32p] * 9)
        lib.lora_oracle_max_threads.restype = ctypes.c_int32
        _lib = lib
    return _lib


def host_cores() -> int:
    """Cores this process may run on."""
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:  # pragma: no cover
        return os.cpu_count() or 1


def _f64(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float64)


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.int32)


def apply(x, y_base, slot_idx, A: Sequence[Optional[np.ndarray]],
          B: Sequence[Optional[np.ndarray]], rank, scale, loaded, threads: int = 1):
    """fp64 LoRA forward.  A[i]: [d_in, r_i], B[i]: [r_i, d_out] (None for empty slots).

    Returns (y [T, d_out] float64, n_invalid).
    """
    lib = _load()
    x = _f64(x)
    yb = _f64(y_base)
    T, d_in = x.shape
    d_out = yb.shape[1]
    assert yb.shape[0] == T
    slot_idx = _i32(slot_idx)
    rank = _i32(rank)
    loaded = _i32(loaded)
    scale = _f64(scale)
    N = rank.shape[0]
    keep = []
    Ap = (_c_f64p * max(N, 1))()
    Bp = (_c_f64p * max(N, 1))()
    for i in range(N):
        if A[i] is None or not loaded[i]:
            Ap[i] = None
            Bp[i] = None
            continue
        a = _f64(A[i])
        b = _f64(B[i])
        assert a.shape == (d_in, rank[i]), (a.shape, d_in, rank[i])
        assert b.shape == (rank[i], d_out), (b.shape, rank[i], d_out)
        keep += [a, b]
        Ap[i] = a.ctypes.data_as(_c_f64p)
        Bp[i] = b.ctypes.data_as(_c_f64p)
    y = np.empty((T, d_out), dtype=np.float64)
    n_inv = lib.lora_oracle_apply(
        T, d_in, d_out, N, x.ctypes.data_as(_c_f64p), d_in, yb.ctypes.data_as(_c_f64p), d_out,
        slot_idx.ctypes.data_as(_c_i32p), Ap, Bp, rank.ctypes.data_as(_c_i32p),
        scale.ctypes.data_as(_c_f64p), loaded.ctypes.data_as(_c_i32p),
        y.ctypes.data_as(_c_f64p), d_out, int(threads))
    if n_inv < 0:
        raise ValueError("lora_oracle_apply: bad argument")
    return y, int(n_inv)


def _widen(h: np.ndarray) -> np.ndarray:
    """bf16 bit patterns -> float64, exactly."""
    h = np.ascontiguousarray(h, dtype=np.uint16)
    return (h.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def apply_workload(wl, call: int = 0, rows: Optional[np.ndarray] = None, threads: int = 1,
                   acts=None):
    """Oracle result for the ``call``-th apply of a workload object.

    ``wl`` is any object with the attributes of
    ``paper_2602_24044_b200.workloads.Workload`` (passed in by the caller; this
    module does not import it).  ``rows`` restricts the evaluation to those
    token rows.  Returns (y float64 [len(rows) or T, d_out], n_invalid).
    """
    target = wl.calls[call]
    x_h, yb_h = acts if acts is not None else wl.activations(call, rows)
    sidx = wl.slot_idx if rows is None else wl.slot_idx[rows]
    N = wl.num_slots
    need = set(int(s) for s in np.unique(sidx) if 0 <= s < N and wl.loaded[s])
    A = [None] * N
    B = [None] * N
    for s in need:
        a_h, b_h = wl.adapter_weights(s, target)
        A[s], B[s] = _widen(a_h), _widen(b_h)
    loaded = np.array([1 if (wl.loaded[i] and i in need) else 0 for i in range(N)], np.int32)
    # slots that are occupied but unused by these rows can stay empty: no row selects them
    return apply(_widen(x_h), _widen(yb_h), sidx, A, B, wl.ranks, wl.scales.astype(np.float64),
                 loaded, threads)


def segment_capacities(T: int, num_slots: int, tile_m: int):
    cap_seg = min(T, num_slots)
    cap_tile = cap_seg + T // tile_m
    return cap_seg, cap_tile


def build_segments(slot_idx, loaded, rank, tile_m: int, long_min: int) -> Dict[str, np.ndarray]:
    """Stable group-by-slot metadata; every array int32, unused entries -1."""
    lib = _load()
    slot_idx = _i32(slot_idx)
    loaded = _i32(loaded)
    rank = _i32(rank)
    T = int(slot_idx.shape[0])
    N = int(rank.shape[0])
    cap_seg, cap_tile = segment_capacities(T, N, tile_m)
    out = {
        "header": np.zeros(5, np.int32),
        "perm": np.empty(T, np.int32),
        "seg_slot": np.empty(cap_seg, np.int32),
        "seg_start": np.empty(cap_seg + 1, np.int32),
        "seg_rank": np.empty(cap_seg, np.int32),
        "seg_flags": np.empty(cap_seg, np.int32),
        "tile_seg": np.empty(cap_tile, np.int32),
        "tile_row0": np.empty(cap_tile, np.int32),
        "tile_rows": np.empty(cap_tile, np.int32),
    }
    p = lambda a: a.ctypes.data_as(_c_i32p)
    rc = lib.lora_oracle_build_segments(
        T, N, p(slot_idx), p(loaded), p(rank), int(tile_m), int(long_min), cap_seg, cap_tile,
        p(out["header"]), p(out["perm"]), p(out["seg_slot"]), p(out["seg_start"]),
        p(out["seg_rank"]), p(out["seg_flags"]), p(out["tile_seg"]), p(out["tile_row0"]),
        p(out["tile_rows"]))
    if rc != 0:
        raise ValueError("lora_oracle_build_segments: bad argument")
    return out
