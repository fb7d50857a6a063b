"""Thin ctypes binding of liblora_b200.so: same names as the C entry points, argument
marshalling only.  Every step of the LoRA forward runs inside the CUDA library; PyTorch is
used by callers for device memory and streams.

The library must have been built (``python -m paper_2602_24044_b200.build``); loading fails
loudly otherwise.  There is no CPU fallback.
"""
from __future__ import annotations

import ctypes
import os
from typing import Dict, Optional, Sequence

import numpy as np

from . import build as _build

LORA_OK = 0
A_DIN_MAJOR = 0
A_RANK_MAJOR = 1
PACKED = 2
META_HEADER_WORDS = 16

EXPORTS = [
    "lora_status_string", "lora_last_cuda_error", "lora_launch_count",
    "lora_pool_bytes", "lora_pool_create", "lora_pool_destroy", "lora_pool_load_slot",
    "lora_pool_evict_slot", "lora_pool_acquire", "lora_pool_read_slot", "lora_pool_slot_info",
    "lora_pool_poll_status", "lora_pool_reset_status", "lora_pool_set_tuning",
    "lora_segments_bytes", "lora_build_segments", "lora_workspace_bytes",
    "lora_bgmv_apply", "lora_sgmv_apply", "lora_apply_host", "lora_bgmv_apply_static",
    "lora_bgmv_apply_multi", "lora_pool_check_status", "lora_pool_selftest_wait_expiry", "lora_pool_plan",
    "lora_policy_create", "lora_policy_destroy", "lora_policy_lookup", "lora_policy_slot",
    "lora_policy_touch", "lora_policy_pin", "lora_policy_unpin", "lora_policy_choose_victim",
    "lora_policy_assign", "lora_policy_release", "lora_policy_admit", "lora_policy_stats",
]
STATIC_SCRATCH_BYTES = 2 * 1024 * 1024


class LoraError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = int(status)
        msg = _lib().lora_status_string(status).decode()
        if status == 9:
            msg += " (cudaError %d)" % _lib().lora_last_cuda_error()
        super().__init__("%s: %s" % (where, msg))


class _Target(ctypes.Structure):
    _fields_ = [("d_in", ctypes.c_int32), ("d_out", ctypes.c_int32)]


class _PoolDesc(ctypes.Structure):
    _fields_ = [("device", ctypes.c_int32), ("num_slots", ctypes.c_int32),
                ("r_max", ctypes.c_int32), ("num_targets", ctypes.c_int32),
                ("targets", ctypes.POINTER(_Target)), ("device_buf", ctypes.c_void_p),
                ("device_buf_bytes", ctypes.c_size_t)]


class _AdapterHost(ctypes.Structure):
    _fields_ = [("rank", ctypes.c_int32), ("scale", ctypes.c_float),
                ("A", ctypes.POINTER(ctypes.c_void_p)), ("B", ctypes.POINTER(ctypes.c_void_p)),
                ("a_layout", ctypes.c_int32), ("trust_pinned", ctypes.c_int32)]


class _ApplyItem(ctypes.Structure):
    _fields_ = [("target", ctypes.c_int32), ("x", ctypes.c_void_p), ("ldx", ctypes.c_int64),
                ("y_base", ctypes.c_void_p), ("ldyb", ctypes.c_int64),
                ("y", ctypes.c_void_p), ("ldy", ctypes.c_int64)]


class _StepBuffers(ctypes.Structure):
    _fields_ = [("x_dev", ctypes.c_void_p), ("y_base_dev", ctypes.c_void_p),
                ("y_dev", ctypes.c_void_p), ("slot_idx_dev", ctypes.c_void_p),
                ("meta_dev", ctypes.c_void_p), ("meta_bytes", ctypes.c_size_t),
                ("workspace", ctypes.c_void_p), ("workspace_bytes", ctypes.c_size_t)]


_handle = None


def library_path() -> str:
    return _build.LIB


def _lib():
    global _handle
    if _handle is None:
        path = library_path()
        if not os.path.exists(path):
            raise RuntimeError(
                "liblora_b200.so is missing (%s): build it with "
                "`python -m paper_2602_24044_b200.build`; there is no fallback path" % path)
        lib = ctypes.CDLL(path)
        lib.lora_status_string.restype = ctypes.c_char_p
        lib.lora_status_string.argtypes = [ctypes.c_int]
        lib.lora_last_cuda_error.restype = ctypes.c_int32
        lib.lora_launch_count.restype = ctypes.c_int64
        vp, i32, i64, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_size_t
        sigs = {
            "lora_pool_bytes": [ctypes.POINTER(_PoolDesc), ctypes.POINTER(sz)],
            "lora_pool_create": [ctypes.POINTER(_PoolDesc), ctypes.POINTER(vp)],
            "lora_pool_destroy": [vp],
            "lora_pool_load_slot": [vp, i32, ctypes.POINTER(_AdapterHost), vp, vp],
            "lora_pool_evict_slot": [vp, i32, vp, vp],
            "lora_pool_acquire": [vp, ctypes.POINTER(i32), i32, vp],
            "lora_pool_read_slot": [vp, i32, i32, vp, vp, vp],
            "lora_pool_slot_info": [vp, i32, ctypes.POINTER(i32), ctypes.POINTER(ctypes.c_float)],
            "lora_pool_poll_status": [vp, vp, vp],
            "lora_pool_reset_status": [vp, vp],
            "lora_pool_set_tuning": [vp, i32, i32],
            "lora_segments_bytes": [i32, i32, i32, ctypes.POINTER(sz)],
            "lora_build_segments": [vp, vp, i32, i32, i32, vp, sz, vp],
            "lora_workspace_bytes": [vp, i32, ctypes.POINTER(sz)],
            "lora_bgmv_apply": [vp, i32, vp, i64, vp, i64, vp, i64, vp, i32, vp, vp, sz, vp],
            "lora_sgmv_apply": [vp, i32, vp, i64, vp, i64, vp, i64, vp, i32, vp, sz, vp],
            "lora_bgmv_apply_static": [vp, i32, vp, i64, vp, i64, vp, i64, vp, i32, vp, vp],
            "lora_apply_host": [vp, i32, i32, vp, vp, vp, vp, i32, i32, i32,
                                ctypes.POINTER(_StepBuffers), vp],
            "lora_bgmv_apply_multi": [vp, ctypes.POINTER(_ApplyItem), i32, vp, i32, vp, vp, sz, vp],
            "lora_pool_check_status": [vp, vp, ctypes.POINTER(i32)],
            "lora_pool_selftest_wait_expiry": [vp, i32, vp, vp],
            "lora_pool_plan": [sz, ctypes.POINTER(_Target), i32, i32, ctypes.POINTER(i32),
                               ctypes.POINTER(sz)],
            "lora_policy_create": [i32, ctypes.POINTER(vp)],
            "lora_policy_destroy": [vp],
            "lora_policy_lookup": [vp, i64, ctypes.POINTER(i32)],
            "lora_policy_slot": [vp, i32, ctypes.POINTER(i64), ctypes.POINTER(i32)],
            "lora_policy_touch": [vp, i32],
            "lora_policy_pin": [vp, ctypes.POINTER(i32), i32],
            "lora_policy_unpin": [vp, ctypes.POINTER(i32), i32],
            "lora_policy_choose_victim": [vp, ctypes.POINTER(i32), ctypes.POINTER(i64)],
            "lora_policy_assign": [vp, i32, i64],
            "lora_policy_release": [vp, i32],
            "lora_policy_admit": [vp, ctypes.POINTER(i64), i32, ctypes.POINTER(i32),
                                  ctypes.POINTER(i32), ctypes.POINTER(i64), i32, ctypes.POINTER(i32)],
            "lora_policy_stats": [vp, ctypes.POINTER(i64), ctypes.POINTER(i64), ctypes.POINTER(i64)],
        }
        for name, args in sigs.items():
            fn = getattr(lib, name)
            fn.restype = ctypes.c_int
            fn.argtypes = args
        _handle = lib
    return _handle


def _check(status: int, where: str) -> None:
    if status != LORA_OK:
        raise LoraError(status, where)


def _ptr(obj) -> Optional[int]:
    """Address of a torch tensor / numpy array / int / None."""
    if obj is None:
        return None
    if isinstance(obj, int):
        return obj
    if hasattr(obj, "data_ptr"):
        return int(obj.data_ptr())
    if isinstance(obj, np.ndarray):
        return int(obj.ctypes.data)
    raise TypeError("cannot take the address of %r" % type(obj))


def _stream(s) -> Optional[int]:
    if s is None:
        return None
    if isinstance(s, int):
        return s
    return int(s.cuda_stream)


def _nbytes(obj) -> int:
    if hasattr(obj, "element_size"):
        return int(obj.numel() * obj.element_size())
    return int(obj.nbytes)


def _desc(num_slots, r_max, targets, device, buf=None, buf_bytes=0):
    arr = (_Target * len(targets))(*[_Target(int(a), int(b)) for a, b in targets])
    d = _PoolDesc(int(device), int(num_slots), int(r_max), len(targets), arr, _ptr(buf),
                  int(buf_bytes))
    d._keep = arr
    return d


# ------------------------------------------------------------------------------------------
# the C entry points
# ------------------------------------------------------------------------------------------
def status_string(status: int) -> str:
    return _lib().lora_status_string(int(status)).decode()


def launch_count() -> int:
    return int(_lib().lora_launch_count())


def pool_bytes(num_slots: int, r_max: int, targets: Sequence, device: int = 0) -> int:
    out = ctypes.c_size_t(0)
    d = _desc(num_slots, r_max, targets, device)
    _check(_lib().lora_pool_bytes(ctypes.byref(d), ctypes.byref(out)), "lora_pool_bytes")
    return int(out.value)


def pool_create(num_slots: int, r_max: int, targets: Sequence, device_buf, device: int = 0,
                device_buf_bytes: Optional[int] = None) -> int:
    out = ctypes.c_void_p(None)
    nbytes = _nbytes(device_buf) if device_buf_bytes is None else device_buf_bytes
    d = _desc(num_slots, r_max, targets, device, device_buf, nbytes)
    _check(_lib().lora_pool_create(ctypes.byref(d), ctypes.byref(out)), "lora_pool_create")
    return int(out.value)


def pool_destroy(pool: int) -> None:
    _check(_lib().lora_pool_destroy(pool), "lora_pool_destroy")


def pool_load_slot(pool: int, slot: int, rank: int, scale: float, A: Sequence, B: Sequence,
                   a_layout: int = A_DIN_MAJOR, load_stream=None, compute_stream=None,
                   trust_pinned: bool = False) -> None:
    n = len(A)
    Ap = (ctypes.c_void_p * n)(*[_ptr(a) for a in A])
    Bp = (ctypes.c_void_p * n)(*[_ptr(b) for b in B])
    ad = _AdapterHost(int(rank), float(scale), Ap, Bp, int(a_layout), int(bool(trust_pinned)))
    _check(_lib().lora_pool_load_slot(pool, int(slot), ctypes.byref(ad), _stream(load_stream),
                                      _stream(compute_stream)), "lora_pool_load_slot")


def pool_evict_slot(pool: int, slot: int, load_stream=None, compute_stream=None) -> None:
    _check(_lib().lora_pool_evict_slot(pool, int(slot), _stream(load_stream),
                                       _stream(compute_stream)), "lora_pool_evict_slot")


def pool_acquire(pool: int, slots: Sequence[int], compute_stream=None) -> None:
    arr = (ctypes.c_int32 * max(len(slots), 1))(*[int(s) for s in slots])
    _check(_lib().lora_pool_acquire(pool, arr, len(slots), _stream(compute_stream)),
           "lora_pool_acquire")


def pool_read_slot(pool: int, slot: int, target: int, A_host, B_host, stream=None) -> None:
    _check(_lib().lora_pool_read_slot(pool, int(slot), int(target), _ptr(A_host), _ptr(B_host),
                                      _stream(stream)), "lora_pool_read_slot")


def pool_slot_info(pool: int, slot: int):
    r = ctypes.c_int32(0)
    s = ctypes.c_float(0)
    _check(_lib().lora_pool_slot_info(pool, int(slot), ctypes.byref(r), ctypes.byref(s)),
           "lora_pool_slot_info")
    return int(r.value), float(s.value)


def pool_poll_status(pool: int, host_out, stream=None) -> None:
    _check(_lib().lora_pool_poll_status(pool, _ptr(host_out), _stream(stream)),
           "lora_pool_poll_status")


def pool_reset_status(pool: int, stream=None) -> None:
    _check(_lib().lora_pool_reset_status(pool, _stream(stream)), "lora_pool_reset_status")


def pool_check_status(pool: int, stream=None):
    """Synchronises `stream`; returns the four status words.  Raises LoraError(10) when a bounded
    device-side wait has expired since the last reset."""
    w = (ctypes.c_int32 * 4)()
    _check(_lib().lora_pool_check_status(pool, _stream(stream), w), "lora_pool_check_status")
    return [int(v) for v in w]


def pool_selftest_wait_expiry(pool: int, polls: int, witness_dev=None, stream=None) -> None:
    _check(_lib().lora_pool_selftest_wait_expiry(pool, int(polls), _ptr(witness_dev),
                                                 _stream(stream)), "lora_pool_selftest_wait_expiry")


def pool_plan(bytes_budget: int, targets: Sequence, r_max: int):
    """(num_slots that fit in bytes_budget, bytes one slot costs)."""
    arr = (_Target * len(targets))(*[_Target(int(a), int(b)) for a, b in targets])
    n, per = ctypes.c_int32(0), ctypes.c_size_t(0)
    _check(_lib().lora_pool_plan(int(bytes_budget), arr, len(targets), int(r_max), ctypes.byref(n),
                                 ctypes.byref(per)), "lora_pool_plan")
    return int(n.value), int(per.value)


# slot policy (host-side bookkeeping, no CUDA call)
def policy_create(num_slots: int) -> int:
    out = ctypes.c_void_p(None)
    _check(_lib().lora_policy_create(int(num_slots), ctypes.byref(out)), "lora_policy_create")
    return int(out.value)


def policy_destroy(policy: int) -> None:
    _check(_lib().lora_policy_destroy(policy), "lora_policy_destroy")


def policy_lookup(policy: int, adapter: int) -> int:
    out = ctypes.c_int32(0)
    _check(_lib().lora_policy_lookup(policy, int(adapter), ctypes.byref(out)), "lora_policy_lookup")
    return int(out.value)


def policy_slot(policy: int, slot: int):
    a, p = ctypes.c_int64(0), ctypes.c_int32(0)
    _check(_lib().lora_policy_slot(policy, int(slot), ctypes.byref(a), ctypes.byref(p)),
           "lora_policy_slot")
    return int(a.value), int(p.value)


def policy_touch(policy: int, slot: int) -> None:
    _check(_lib().lora_policy_touch(policy, int(slot)), "lora_policy_touch")


def _i32_array(values):
    return (ctypes.c_int32 * max(len(values), 1))(*[int(v) for v in values])


def policy_pin(policy: int, slots: Sequence[int]) -> None:
    _check(_lib().lora_policy_pin(policy, _i32_array(slots), len(slots)), "lora_policy_pin")


def policy_unpin(policy: int, slots: Sequence[int]) -> None:
    _check(_lib().lora_policy_unpin(policy, _i32_array(slots), len(slots)), "lora_policy_unpin")


def policy_choose_victim(policy: int):
    """(slot, adapter it holds now or -1)."""
    s, a = ctypes.c_int32(0), ctypes.c_int64(0)
    _check(_lib().lora_policy_choose_victim(policy, ctypes.byref(s), ctypes.byref(a)),
           "lora_policy_choose_victim")
    return int(s.value), int(a.value)


def policy_assign(policy: int, slot: int, adapter: int) -> None:
    _check(_lib().lora_policy_assign(policy, int(slot), int(adapter)), "lora_policy_assign")


def policy_release(policy: int, slot: int) -> None:
    _check(_lib().lora_policy_release(policy, int(slot)), "lora_policy_release")


def policy_admit(policy: int, adapters: Sequence[int], miss_cap: Optional[int] = None):
    """(slot_idx int32 array, [(slot, adapter) to load, ...]) for one batch of requests."""
    n = len(adapters)
    cap = n if miss_cap is None else int(miss_cap)
    ids = (ctypes.c_int64 * max(n, 1))(*[int(a) for a in adapters])
    sidx = (ctypes.c_int32 * max(n, 1))()
    ms = (ctypes.c_int32 * max(cap, 1))()
    ma = (ctypes.c_int64 * max(cap, 1))()
    nm = ctypes.c_int32(0)
    _check(_lib().lora_policy_admit(policy, ids, n, sidx, ms, ma, cap, ctypes.byref(nm)),
           "lora_policy_admit")
    return (np.array(sidx[:n], dtype=np.int32),
            [(int(ms[k]), int(ma[k])) for k in range(nm.value)])


def policy_stats(policy: int):
    h, m, e = ctypes.c_int64(0), ctypes.c_int64(0), ctypes.c_int64(0)
    _check(_lib().lora_policy_stats(policy, ctypes.byref(h), ctypes.byref(m), ctypes.byref(e)),
           "lora_policy_stats")
    return int(h.value), int(m.value), int(e.value)


def pool_set_tuning(pool: int, key: int, value: int) -> None:
    _check(_lib().lora_pool_set_tuning(pool, int(key), int(value)), "lora_pool_set_tuning")


def segments_bytes(T: int, num_slots: int, tile_m: int) -> int:
    out = ctypes.c_size_t(0)
    _check(_lib().lora_segments_bytes(int(T), int(num_slots), int(tile_m), ctypes.byref(out)),
           "lora_segments_bytes")
    return int(out.value)


def build_segments(pool: int, slot_idx_dev, T: int, tile_m: int, long_min: int, meta_dev,
                   meta_bytes: Optional[int] = None, stream=None) -> None:
    nbytes = _nbytes(meta_dev) if meta_bytes is None else meta_bytes
    _check(_lib().lora_build_segments(pool, _ptr(slot_idx_dev), int(T), int(tile_m), int(long_min),
                                      _ptr(meta_dev), nbytes, _stream(stream)),
           "lora_build_segments")


def workspace_bytes(pool: int, T_max: int) -> int:
    out = ctypes.c_size_t(0)
    _check(_lib().lora_workspace_bytes(pool, int(T_max), ctypes.byref(out)), "lora_workspace_bytes")
    return int(out.value)


def bgmv_apply(pool: int, target: int, x, ldx: int, y_base, ldyb: int, y, ldy: int, slot_idx_dev,
               T: int, meta_dev, workspace, workspace_bytes_: Optional[int] = None,
               stream=None) -> None:
    nbytes = (_nbytes(workspace) if workspace is not None else 0) \
        if workspace_bytes_ is None else workspace_bytes_
    _check(_lib().lora_bgmv_apply(pool, int(target), _ptr(x), int(ldx), _ptr(y_base), int(ldyb),
                                  _ptr(y), int(ldy), _ptr(slot_idx_dev), int(T), _ptr(meta_dev),
                                  _ptr(workspace), nbytes, _stream(stream)), "lora_bgmv_apply")


def make_apply_items(items: Sequence):
    """items: (target, x, ldx, y_base, ldyb, y, ldy) tuples -> a C array for bgmv_apply_multi (build
    it once when the same launch is issued repeatedly)."""
    arr = (_ApplyItem * max(len(items), 1))()
    for k, (target, x, ldx, yb, ldyb, y, ldy) in enumerate(items):
        arr[k] = _ApplyItem(int(target), _ptr(x), int(ldx), _ptr(yb), int(ldyb), _ptr(y), int(ldy))
    return arr, len(items)


def bgmv_apply_multi(pool: int, items, slot_idx_dev, T: int, meta_dev, workspace,
                     workspace_bytes_: Optional[int] = None, stream=None) -> None:
    """Several projections of one decode batch in one launch; `items` as for make_apply_items (or
    its result)."""
    arr, n = items if isinstance(items, tuple) and len(items) == 2 and not isinstance(items[0], tuple) \
        else make_apply_items(items)
    nbytes = (_nbytes(workspace) if workspace is not None else 0) \
        if workspace_bytes_ is None else workspace_bytes_
    _check(_lib().lora_bgmv_apply_multi(pool, arr, n, _ptr(slot_idx_dev), int(T), _ptr(meta_dev),
                                        _ptr(workspace), nbytes, _stream(stream)),
           "lora_bgmv_apply_multi")


def bgmv_apply_static(pool: int, target: int, x, ldx: int, y_base, ldyb: int, y, ldy: int,
                      slot_idx_dev, T: int, meta_dev, stream=None) -> None:
    """lora_bgmv_apply without a workspace argument: the scratch is a fixed array inside the
    library (for callers that must not allocate device memory).  See lora_b200.h for the size
    limit and the rule about overlapping calls."""
    _check(_lib().lora_bgmv_apply_static(pool, int(target), _ptr(x), int(ldx), _ptr(y_base),
                                         int(ldyb), _ptr(y), int(ldy), _ptr(slot_idx_dev), int(T),
                                         _ptr(meta_dev), _stream(stream)), "lora_bgmv_apply_static")


def sgmv_apply(pool: int, target: int, x, ldx: int, y_base, ldyb: int, y, ldy: int, meta_dev,
               T: int, workspace, workspace_bytes_: Optional[int] = None, stream=None) -> None:
    nbytes = (_nbytes(workspace) if workspace is not None else 0) \
        if workspace_bytes_ is None else workspace_bytes_
    _check(_lib().lora_sgmv_apply(pool, int(target), _ptr(x), int(ldx), _ptr(y_base), int(ldyb),
                                  _ptr(y), int(ldy), _ptr(meta_dev), int(T), _ptr(workspace),
                                  nbytes, _stream(stream)), "lora_sgmv_apply")


def apply_host(pool: int, target: int, kind: int, x_host, y_base_host, y_host, slot_idx_host,
               T: int, tile_m: int, long_min: int, x_dev, y_base_dev, y_dev, slot_idx_dev,
               meta_dev, workspace, stream=None) -> None:
    sb = _StepBuffers(_ptr(x_dev), _ptr(y_base_dev), _ptr(y_dev), _ptr(slot_idx_dev),
                      _ptr(meta_dev), _nbytes(meta_dev), _ptr(workspace), _nbytes(workspace))
    _check(_lib().lora_apply_host(pool, int(target), int(kind), _ptr(x_host), _ptr(y_base_host),
                                  _ptr(y_host), _ptr(slot_idx_host), int(T), int(tile_m),
                                  int(long_min), ctypes.byref(sb), _stream(stream)),
           "lora_apply_host")


# ------------------------------------------------------------------------------------------
# reading a metadata buffer copied back to the host
# ------------------------------------------------------------------------------------------
def unpack_segments(meta: np.ndarray, T: int, num_slots: int, tile_m: int) -> Dict[str, np.ndarray]:
    """Split the int32 words of a metadata buffer into its named arrays (see lora_b200.h)."""
    meta = np.asarray(meta, dtype=np.int32)
    cap_seg = min(T, num_slots)
    cap_tile = cap_seg + T // tile_m
    out: Dict[str, np.ndarray] = {"header_full": meta[:META_HEADER_WORDS].copy()}
    out["header"] = meta[:5].copy()
    o = META_HEADER_WORDS
    for name, n in [("perm", T), ("seg_slot", cap_seg), ("seg_start", cap_seg + 1),
                    ("seg_rank", cap_seg), ("seg_flags", cap_seg), ("tile_seg", cap_tile),
                    ("tile_row0", cap_tile), ("tile_rows", cap_tile), ("tile_flags", cap_tile)]:
        out[name] = meta[o:o + n].copy()
        o += n
    o = (o + 3) & ~3
    out["tile_desc"] = meta[o:o + 4 * cap_tile].reshape(cap_tile, 4).copy()   # library-private
    return out
