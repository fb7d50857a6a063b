"""Host-only checks of the C-ABI library: it builds for sm_100a, loads without a GPU, exports
every symbol the public header declares, and rejects bad arguments before touching a device."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_2602_24044_b200 import binding as lb
from paper_2602_24044_b200 import build as lbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    lbuild.build()
    return ctypes.CDLL(lbuild.LIB)


def _declared_symbols():
    names = set()
    inc = os.path.join(ROOT, "include")
    for fn in os.listdir(inc):
        if fn.endswith(".h"):
            text = open(os.path.join(inc, fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(lora_[a-z0-9_]+)\s*\(", text))
    return names


def test_every_declared_symbol_is_exported(lib):
    declared = _declared_symbols()
    assert {"lora_pool_create", "lora_pool_load_slot", "lora_build_segments", "lora_bgmv_apply",
            "lora_sgmv_apply"} <= declared
    for name in declared:
        assert hasattr(lib, name), name
    assert set(lb.EXPORTS) <= declared


def test_status_strings():
    assert lb.status_string(0) == "ok"
    seen = {lb.status_string(i) for i in range(11)}   # every code has its own text
    assert len(seen) == 11 and "unknown status" not in seen
    assert lb.status_string(99) == "unknown status"


def test_pool_bytes_and_shape_validation():
    # 128 slots x rank 16 x (4096 + 4096) bf16 = 33.5 MB of weights + a small control block
    n = lb.pool_bytes(128, 16, [(4096, 4096)])
    weights = 128 * 16 * 8192 * 2
    assert weights < n < weights + 1024 * 1024
    # Llama-3-8B, 7 projections x 32 layers, rank 16: 83.9 MB per adapter
    t = [(4096, 4096), (4096, 1024), (4096, 1024), (4096, 4096), (4096, 14336), (4096, 14336),
         (14336, 4096)] * 32
    per_adapter = (lb.pool_bytes(2, 16, t) - lb.pool_bytes(1, 16, t))
    assert per_adapter == 16 * 2 * sum(a + b for a, b in t) == 83886080
    for bad, status in [(dict(num_slots=0), 1), (dict(r_max=0), 4), (dict(r_max=65), 4),
                        (dict(targets=[(4100, 4096)]), 2), (dict(targets=[(4096, 0)]), 2)]:
        kw = dict(num_slots=4, r_max=8, targets=[(64, 64)])
        kw.update(bad)
        with pytest.raises(lb.LoraError) as e:
            lb.pool_bytes(**kw)
        assert e.value.status == status


def test_pool_create_rejects_bad_buffers_before_any_device_call():
    buf = np.zeros(1 << 20, np.uint8)
    aligned = buf.ctypes.data + (-buf.ctypes.data) % 256
    with pytest.raises(lb.LoraError) as e:          # misaligned
        lb.pool_create(4, 8, [(64, 64)], aligned + 8, device_buf_bytes=1 << 19)
    assert e.value.status == 1
    with pytest.raises(lb.LoraError) as e:          # too small
        lb.pool_create(4, 8, [(64, 64)], aligned, device_buf_bytes=128)
    assert e.value.status == 7


def test_segments_bytes_matches_documented_layout():
    T, N, tile_m = 256, 128, 16
    cap_seg, cap_tile = min(T, N), min(T, N) + T // tile_m
    words = 16 + T + 4 * cap_seg + 1 + 4 * cap_tile
    public_words = words
    words = (words + 3) // 4 * 4 + 4 * cap_tile          # library-private tile records
    desc_end = words
    cap_unit = cap_tile * ((tile_m + 15) // 16)          # 16-row pieces of all tiles
    words += 4 * cap_unit + 16 * cap_unit                # library-private unit records and row ids
    words += (cap_tile + 1 + 3) // 4 * 4                 # library-private list of long tiles
    assert lb.segments_bytes(T, N, tile_m) == 4 * words
    assert lb.segments_bytes(0, N, tile_m) == 4 * 24      # header, seg_start[1], padding, list count
    with pytest.raises(lb.LoraError):
        lb.segments_bytes(-1, N, tile_m)
    meta = np.arange(words, dtype=np.int32)
    parts = lb.unpack_segments(meta, T, N, tile_m)
    assert parts["perm"][0] == 16 and len(parts["tile_flags"]) == cap_tile
    assert parts["tile_flags"][-1] == public_words - 1
    assert parts["tile_desc"][-1, -1] == desc_end - 1


def test_null_handles_are_rejected():
    for call in (lambda: lb.pool_destroy(None), lambda: lb.workspace_bytes(None, 8),
                 lambda: lb.pool_set_tuning(None, 0, 0),
                 lambda: lb.build_segments(None, 0, 4, 16, 128, 0, meta_bytes=0)):
        with pytest.raises(lb.LoraError) as e:
            call()
        assert e.value.status == 1


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(lb, "_handle", None)
    monkeypatch.setattr(lb, "library_path", lambda: str(tmp_path / "absent.so"))
    with pytest.raises(RuntimeError, match="no fallback"):
        lb.launch_count()
