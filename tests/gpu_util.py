"""Helpers shared by the GPU parity tests."""
import numpy as np
import pytest

from oracle import lora_oracle as orc
from paper_2602_24044_b200 import workloads as W


def require_gpu():
    import torch
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2602_24044_b200 import build as lbuild
    lbuild.build()


def check_tolerance(y_bits: np.ndarray, y_ref: np.ndarray, tight: bool = True, what: str = ""):
    """The stated bound |y - y_ref| <= 1e-2 |y_ref| + 1e-2 on every element, plus (tight) the
    bound the arithmetic supports: half a bf16 ulp of the result and fp32 accumulation noise."""
    y = W.bf16_to_f64(y_bits)
    err = np.abs(y - y_ref)
    bound = 1e-2 * np.abs(y_ref) + 1e-2
    bad = err > bound
    assert not bad.any(), "%s: %d elements outside the stated tolerance, worst %.3g at %s" % (
        what, int(bad.sum()), float((err - bound).max()), np.unravel_index(np.argmax(err - bound), err.shape))
    if tight:
        tb = 2.0 ** -8 * np.abs(y_ref) * 1.002 + 2e-4
        worst = float((err - tb).max())
        assert worst <= 0, "%s: error exceeds half a bf16 ulp + 2e-4 by %.3g" % (what, worst)
    return float(err.max())


def oracle_full(wl, call=0, threads=8):
    return orc.apply_workload(wl, call, threads=threads)


ARRAYS = ["header", "perm", "seg_slot", "seg_start", "seg_rank", "seg_flags",
          "tile_seg", "tile_row0", "tile_rows"]


def check_segments(got: dict, wl, tile_m, long_min, slot_idx=None, loaded=None):
    sidx = wl.slot_idx if slot_idx is None else slot_idx
    ld = wl.loaded if loaded is None else loaded
    ref = orc.build_segments(sidx, ld, wl.ranks, tile_m, long_min)
    for name in ARRAYS:
        assert np.array_equal(got[name], ref[name]), name
    # private per-tile flag: rows of the tile are consecutive token ids
    n_tile = ref["header"][4]
    for k in range(n_tile):
        r0, rows = ref["tile_row0"][k], ref["tile_rows"][k]
        p = ref["perm"][r0:r0 + rows]
        assert got["tile_flags"][k] == int(np.all(np.diff(p) == 1)), k
    assert np.all(got["tile_flags"][n_tile:] == -1)
    return ref
