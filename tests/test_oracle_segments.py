"""Pins for the oracle's segment metadata (stable group-by-slot), CPU only."""
import numpy as np
import pytest

from conftest import read_golden
from oracle import lora_oracle as orc
from paper_2602_24044_b200 import workloads as W

ARRAYS = ["header", "perm", "seg_slot", "seg_start", "seg_rank", "seg_flags",
          "tile_seg", "tile_row0", "tile_rows"]


def test_hand_worked_example():
    g = read_golden("segments_hand.txt")
    ints = lambda k: np.array(g[k], np.int32)
    out = orc.build_segments(ints("slot_idx"), ints("loaded"), ints("rank"),
                             int(g["tile_m"][0]), int(g["long_min"][0]))
    for name in ARRAYS:
        assert np.array_equal(out[name], ints(name)), name


def _library_reference(slot_idx, loaded, rank, tile_m, long_min):
    """Same metadata from numpy's stable argsort and unique (library routines)."""
    T, N = len(slot_idx), len(rank)
    inr = (slot_idx >= 0) & (slot_idx < N)
    active = inr.copy()
    active[inr] = loaded[slot_idx[inr]] != 0
    act_t = np.nonzero(active)[0]
    order = act_t[np.argsort(slot_idx[act_t], kind="stable")]
    perm = np.concatenate([order, np.nonzero(~active)[0]]).astype(np.int32)
    slots, starts, counts = np.unique(slot_idx[order], return_index=True, return_counts=True)
    flags, tiles = [], []
    for s, (st, c) in enumerate(zip(starts, counts)):
        rows = order[st:st + c]
        contiguous = int(np.all(np.diff(rows) == 1))
        flags.append(contiguous | (2 if c >= long_min else 0))
        for r0 in range(st, st + c, tile_m):
            tiles.append((s, r0, min(tile_m, st + c - r0)))
    header = [T, len(order), int(np.sum(~active & (slot_idx != -1))), len(slots), len(tiles)]
    return header, perm, slots, np.append(starts, len(order)), rank[slots], flags, tiles


@pytest.mark.parametrize("seed", range(6))
@pytest.mark.parametrize("tile_m", [1, 16, 128])
def test_random_tables_match_library_sort(seed, tile_m):
    rng = np.random.default_rng(seed)
    T = int(rng.integers(1, 700))
    N = int(rng.integers(1, 50))
    slot_idx = rng.integers(-2, N + 2, T).astype(np.int32)
    if seed % 2:
        slot_idx = np.repeat(slot_idx[: max(1, T // 40)], 40)[:T]     # long runs
        T = len(slot_idx)
    loaded = (rng.random(N) < 0.8).astype(np.int32)
    rank = rng.integers(1, 65, N).astype(np.int32)
    out = orc.build_segments(slot_idx, loaded, rank, tile_m, 64)
    header, perm, slots, starts, ranks, flags, tiles = _library_reference(
        slot_idx, loaded, rank, tile_m, 64)
    n_seg, n_tile = header[3], header[4]
    assert list(out["header"]) == header
    assert np.array_equal(out["perm"], perm)
    assert np.array_equal(out["seg_slot"][:n_seg], slots)
    assert np.array_equal(out["seg_start"][:n_seg + 1], starts)
    assert np.array_equal(out["seg_rank"][:n_seg], ranks)
    assert list(out["seg_flags"][:n_seg]) == flags
    got_tiles = list(zip(out["tile_seg"][:n_tile], out["tile_row0"][:n_tile],
                         out["tile_rows"][:n_tile]))
    assert got_tiles == tiles
    for name in ["seg_slot", "seg_rank", "seg_flags"]:
        assert np.all(out[name][n_seg:] == -1)
    assert np.all(out["seg_start"][n_seg + 1:] == -1)
    for name in ["tile_seg", "tile_row0", "tile_rows"]:
        assert np.all(out[name][n_tile:] == -1)


@pytest.mark.parametrize("cfg", [0, 1, 2, 3, 4])
def test_invariants_on_configs(cfg):
    wl = W.make_config(cfg, layers=1)
    out = orc.build_segments(wl.slot_idx, wl.loaded, wl.ranks, wl.tile_m, wl.long_min)
    T, n_active, n_invalid, n_seg, n_tile = out["header"]
    assert T == wl.T and n_invalid == 0 and n_active == T
    assert np.array_equal(np.sort(out["perm"]), np.arange(T))
    ss = out["seg_slot"][:n_seg]
    assert np.all(np.diff(ss) > 0)
    st = out["seg_start"][:n_seg + 1]
    assert st[0] == 0 and st[-1] == n_active and np.all(np.diff(st) > 0)
    for s in range(n_seg):
        assert np.all(wl.slot_idx[out["perm"][st[s]:st[s + 1]]] == ss[s])
        assert np.all(np.diff(out["perm"][st[s]:st[s + 1]]) > 0)        # stable
    # tiles partition the segments in order
    pos = 0
    for k in range(n_tile):
        s, r0, rows = out["tile_seg"][k], out["tile_row0"][k], out["tile_rows"][k]
        assert r0 == pos and 1 <= rows <= wl.tile_m and r0 + rows <= st[s + 1] and r0 >= st[s]
        pos += rows
    assert pos == n_active
    assert n_seg == len(wl.distinct_slots())


def test_degenerate_batches():
    rank = np.full(4, 8, np.int32)
    ld = np.ones(4, np.int32)
    e = orc.build_segments(np.zeros(0, np.int32), ld, rank, 16, 128)
    assert list(e["header"]) == [0, 0, 0, 0, 0] and e["seg_start"][0] == 0
    none = orc.build_segments(np.full(5, -1, np.int32), ld, rank, 16, 128)
    assert list(none["header"]) == [5, 0, 0, 0, 0]
    assert np.array_equal(none["perm"], np.arange(5))
    one = orc.build_segments(np.array([3], np.int32), ld, rank, 16, 1)
    assert list(one["header"]) == [1, 1, 0, 1, 1] and one["seg_flags"][0] == 3
    same = orc.build_segments(np.full(40, 2, np.int32), ld, rank, 16, 32)
    assert list(same["header"]) == [40, 40, 0, 1, 3]
    assert list(same["tile_rows"][:3]) == [16, 16, 8] and same["seg_flags"][0] == 3
    distinct = orc.build_segments(np.array([3, 1, 2, 0], np.int32), ld, rank, 16, 128)
    assert list(distinct["perm"]) == [3, 1, 2, 0] and distinct["header"][3] == 4


def test_workload_generators_are_seeded_and_shaped():
    a, b = W.make_config(1), W.make_config(1)
    assert np.array_equal(a.slot_idx, b.slot_idx)
    assert np.array_equal(a.activations(0)[0], b.activations(0)[0])
    assert np.array_equal(a.adapter_weights(5, 0)[1], b.adapter_weights(5, 0)[1])
    assert not np.array_equal(a.slot_idx, W.make_config(1, rep=1).slot_idx)
    assert 50 <= len(a.distinct_slots()) <= 85                       # Zipf(1.1) over 128 slots
    c2 = W.make_config(2)
    assert 12000 <= c2.T <= 40000 and set(np.unique(c2.ranks)) <= {8, 16, 32}
    c3 = W.make_config(3)
    assert c3.T == 2560 and c3.targets == [(4096, 6144)]
    c4 = W.make_config(4)
    assert len(c4.calls) == 224 and not set(c4.swap_victims) & set(c4.slot_idx.tolist())
    # bf16 rounding is round-to-nearest-even and exact on representable values
    v = np.array([1.0, 1.00390625, 1.01171875, -2.5, 3.140625], np.float32)
    assert np.array_equal(W.bf16_to_f32(W.bf16_round(v)),
                          np.array([1.0, 1.0, 1.015625, -2.5, 3.140625], np.float32))
