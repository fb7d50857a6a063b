"""GPU parity: the CUDA library (through its C ABI) against the fp64 oracle, element by element,
on the same seeded inputs; integer metadata bit-exact."""
import numpy as np
import pytest

from gpu_util import check_segments, check_tolerance, oracle_full, require_gpu
from oracle import lora_oracle as orc
from paper_2602_24044_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _gpu():
    require_gpu()


def _session(wl, **kw):
    from paper_2602_24044_b200.harness import Session
    return Session(wl, **kw)


def _bits(t):
    from paper_2602_24044_b200.harness import bf16_bits
    return bf16_bits(t)


# ---------------------------------------------------------------------------------------------
# segment metadata: bit-exact
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("tile_m", [1, 16, 128])
@pytest.mark.parametrize("case", ["random", "same", "distinct", "none", "invalid", "sorted",
                                  "T0", "T1", "ragged"])
def test_segments_bit_exact(case, tile_m):
    kw = dict(T=333, d_in=64, d_out=64, num_slots=37, ranks=[8, 16, 4, 32], unloaded=(3, 11))
    if case == "random":
        kw.update(index="uniform", frac_none=0.1)
    elif case == "same":
        kw.update(index="same")
    elif case == "distinct":
        kw.update(index="distinct", T=37)
    elif case == "none":
        kw.update(frac_none=1.0)
    elif case == "invalid":
        kw.update(frac_invalid=0.3, frac_none=0.1)
    elif case == "sorted":
        kw.update(index="sorted")
    elif case == "T0":
        kw.update(T=0)
    elif case == "T1":
        kw.update(T=1)
    elif case == "ragged":
        kw.update(T=1001, index="zipf")
    wl = W.make_custom(**kw)
    with _session(wl) as s:
        s.build_segments(tile_m=tile_m, long_min=64)
        got = s.segments_host()
        ref = check_segments(got, wl, tile_m, 64)
        assert s.status()[0] == ref["header"][2]


@pytest.mark.parametrize("tile_m", [1, 16, 100, 128])
@pytest.mark.parametrize("case", ["uniform", "sorted", "zipf", "invalid", "same", "none"])
def test_segments_bit_exact_long_batches(case, tile_m):
    """Batches of 1024 tokens and more take the chunk-parallel builder: same table, bit for bit."""
    kw = dict(T=4999, d_in=64, d_out=64, num_slots=53, ranks=[8, 16, 4, 32], unloaded=(5, 17))
    if case == "uniform":
        kw.update(index="uniform", frac_none=0.05, T=1024)
    elif case == "sorted":
        kw.update(index="sorted")
    elif case == "zipf":
        kw.update(index="zipf", T=7777)
    elif case == "invalid":
        kw.update(frac_invalid=0.2, frac_none=0.2, T=3001)
    elif case == "same":
        kw.update(index="same", T=2048)
    elif case == "none":
        kw.update(frac_none=1.0, T=1500)
    wl = W.make_custom(**kw)
    with _session(wl) as s:
        s.build_segments(tile_m=tile_m, long_min=64)
        got = s.segments_host()
        ref = check_segments(got, wl, tile_m, 64)
        assert s.status()[0] == ref["header"][2]


@pytest.mark.parametrize("cfg", [0, 1, 2, 3, 4])
def test_segments_on_configs(cfg):
    # config 4: one layer's pool is enough, the token list does not depend on the layer count
    wl = W.make_config(cfg, layers=1) if cfg == 4 else W.make_config(cfg)
    with _session(wl, slots=[]) as s:
        # an empty pool first: every token is invalid
        s.build_segments()
        got = s.segments_host()
        check_segments(got, wl, wl.tile_m, wl.long_min, loaded=np.zeros(wl.num_slots, np.int32))
    # slot table only (no weights needed): load rank/scale through tiny single-target pools
    small = W.make_custom(wl.T, 8, 8, wl.num_slots, wl.ranks, r_max=wl.r_max, slot_idx=wl.slot_idx,
                          tile_m=wl.tile_m, long_min=wl.long_min)
    with _session(small) as s:
        s.build_segments()
        check_segments(s.segments_host(), small, wl.tile_m, wl.long_min)


# ---------------------------------------------------------------------------------------------
# pool round trip
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("a_layout", [0, 1])
def test_pool_round_trip(a_layout):
    wl = W.make_custom(8, 264, 136, 5, [1, 7, 8, 12, 16], r_max=16)
    with _session(wl, a_layout=a_layout) as s:
        for slot in range(5):
            A_h, B_h = wl.adapter_weights(slot, 0)
            r = int(wl.ranks[slot])
            A_d, B_d = s.read_slot(slot, 0)
            assert np.array_equal(A_d[:r], A_h.T)
            assert np.array_equal(B_d[:r], B_h)
            assert not A_d[r:].any() and not B_d[r:].any()       # padding rows are zero
        # overwrite slot 4 (rank 16) with the rank-1 adapter: stale rows must be cleared
        s.load_slot(4, a_layout=a_layout, src_slot=0)
        import torch
        torch.cuda.synchronize()
        A_d, B_d = s.read_slot(4, 0)
        A_h, B_h = wl.adapter_weights(0, 0)
        assert np.array_equal(A_d[:1], A_h.T) and not A_d[1:].any() and not B_d[1:].any()


# ---------------------------------------------------------------------------------------------
# the forward
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("grouped", [True, False])
@pytest.mark.parametrize("rank", [1, 8, 16, 32, 64])
@pytest.mark.parametrize("T", [1, 15, 16, 17, 70])
def test_bgmv_small_shapes(T, rank, grouped):
    wl = W.make_custom(T, 264, 520, 6, rank, scale=0.3, frac_none=0.15, frac_invalid=0.1,
                       unloaded=(2,), weight_mode="unitB", seed=T * 100 + rank)
    y_ref, n_inv = oracle_full(wl)
    with _session(wl) as s:
        y = s.apply(grouped=grouped)
        check_tolerance(_bits(y), y_ref, what="bgmv T=%d r=%d" % (T, rank))
        assert s.status()[0] == n_inv
        # tokens without an adapter are a bit copy of y_base
        _, yb_h = wl.activations(0)
        idle = ~wl.active_mask()
        assert np.array_equal(_bits(y)[idle], yb_h[idle])


def test_bgmv_empty_batch():
    wl = W.make_custom(0, 64, 64, 4, 8)
    with _session(wl) as s:
        import torch
        x = torch.empty((0, 64), dtype=torch.bfloat16, device=s.device)
        y = s.apply(x=x, y_base=torch.empty_like(x), grouped=False)
        assert y.shape[0] == 0


@pytest.mark.parametrize("grouped", [True, False])
def test_mixed_ranks_and_delta_isolation(grouped):
    """y_base = 0 and B ~ N(0,1): the whole result is the adapter term, so the relative part
    of the tolerance applies to it."""
    wl = W.make_custom(200, 1024, 768, 40, [1, 3, 8, 9, 16, 24, 32, 40, 64], scale=[0.3, 1.7, 2.0],
                       index="zipf", weight_mode="unitB", act_mode="zero_base", tile_m=16)
    y_ref, _ = oracle_full(wl)
    with _session(wl) as s:
        y = s.apply(grouped=grouped)
        check_tolerance(_bits(y), y_ref, what="delta isolation")


@pytest.mark.parametrize("grouped", [True, False])
@pytest.mark.parametrize("in_place", [True, False])
def test_exact_integer_case_is_bit_exact(grouped, in_place):
    """Small-integer inputs: every intermediate is exact in fp32 and the result fits bf16, so
    the GPU must reproduce the oracle bit for bit."""
    wl = W.make_custom(100, 2048, 1032, 9, [1, 4, 8, 16, 32], scale=2.0, weight_mode="int",
                       act_mode="int", frac_none=0.1)
    y_ref, _ = oracle_full(wl)
    assert np.abs(y_ref).max() < 256 and np.all(y_ref == np.rint(y_ref))
    with _session(wl) as s:
        y = s.apply(grouped=grouped, in_place=in_place)
        assert np.array_equal(W.bf16_to_f64(_bits(y)), y_ref)


def test_rerun_and_permutation_are_bit_identical():
    import torch
    wl = W.make_custom(256, 1024, 1024, 32, [8, 16], scale=0.7, index="zipf", frac_none=0.05)
    x_h, yb_h = wl.activations(0)
    rng = np.random.default_rng(0)
    p = rng.permutation(wl.T)
    with _session(wl) as s:
        from paper_2602_24044_b200.harness import bf16_tensor
        y1 = _bits(s.apply())
        y2 = _bits(s.apply())
        assert np.array_equal(y1, y2)
        yt = _bits(s.apply(grouped=False))
        sp = torch.from_numpy(np.ascontiguousarray(wl.slot_idx[p])).to(s.device)
        yp = _bits(s.apply(x=bf16_tensor(x_h[p], s.device), y_base=bf16_tensor(yb_h[p], s.device),
                           slot_idx_dev=sp))
        assert np.array_equal(yp, y1[p])
        ypt = _bits(s.apply(x=bf16_tensor(x_h[p], s.device), y_base=bf16_tensor(yb_h[p], s.device),
                            slot_idx_dev=sp, grouped=False))
        assert np.array_equal(ypt, yt[p])


def test_strided_inputs_and_in_place():
    import torch
    from paper_2602_24044_b200.harness import bf16_tensor
    wl = W.make_custom(40, 512, 256, 4, 16, scale=1.1)
    y_ref, _ = oracle_full(wl)
    x_h, yb_h = wl.activations(0)
    with _session(wl) as s:
        xw = torch.zeros((40, 512 + 64), dtype=torch.bfloat16, device=s.device)
        xw[:, :512] = bf16_tensor(x_h, s.device)
        ybw = torch.zeros((40, 256 + 8), dtype=torch.bfloat16, device=s.device)
        ybw[:, :256] = bf16_tensor(yb_h, s.device)
        y = s.apply(x=xw[:, :512], y_base=ybw[:, :256], in_place=True)
        assert y.data_ptr() == ybw.data_ptr()
        check_tolerance(_bits(ybw[:, :256]), y_ref, what="strided in place")
        assert not _bits(ybw[:, 256:]).any()


@pytest.mark.parametrize("cfg", [0, 1])
@pytest.mark.parametrize("grouped", [True, False])
def test_decode_configs(cfg, grouped):
    wl = W.make_config(cfg)
    y_ref, n_inv = oracle_full(wl)
    with _session(wl) as s:
        y = s.apply(grouped=grouped)
        check_tolerance(_bits(y), y_ref, what="config %d" % cfg)
        assert s.status()[0] == 0 == n_inv


def test_mixed_chunked_prefill_config():
    wl = W.make_config(3)
    y_ref, _ = oracle_full(wl)
    with _session(wl) as s:
        y = s.apply()
        check_tolerance(_bits(y), y_ref, what="config 3")


def test_prefill_config_every_row():
    """Config 2 at full size, both projections, in the launch configuration the benchmark times:
    EVERY row of the GPU result against the oracle (the oracle goes through the batch in blocks of
    rows so that its fp64 copies stay small), with the tight bound."""
    from paper_2602_24044_b200.harness import bf16_tensor
    wl = W.make_config(2)
    threads = orc.host_cores()
    with _session(wl) as s:
        for call in (0, 1):
            x_h, yb_h = wl.activations(call)
            y = _bits(s.apply(call, x=bf16_tensor(x_h, s.device), y_base=bf16_tensor(yb_h, s.device)))
            assert s.status()[1] == 0
            for r0 in range(0, wl.T, 2048):
                rows = np.arange(r0, min(wl.T, r0 + 2048))
                y_ref, _ = orc.apply_workload(wl, call, rows=rows, threads=threads,
                                              acts=(x_h[rows], yb_h[rows]))
                check_tolerance(y[rows], y_ref, what="config 2 call %d rows %d.." % (call, r0))


def test_layer_step_config_all_projections():
    """Config 4 restricted to one layer's seven projections (the other layers repeat the same
    shapes with other seeds)."""
    wl = W.make_config(4, layers=1)
    with _session(wl) as s:
        for call in range(7):
            y_ref, _ = oracle_full(wl, call)
            y = s.apply(call, rebuild=(call == 0))
            check_tolerance(_bits(y), y_ref, what="config 4 projection %d" % call)


def test_back_to_back_applies_on_one_table():
    """Several applies queued behind one metadata build, without a host synchronisation between
    them: from the second on, the kernels may read the table and the pool before their predecessor
    has finished (programmatic dependent launch).  Every result must still match the oracle."""
    from paper_2602_24044_b200 import binding as lb
    from paper_2602_24044_b200.harness import bf16_tensor
    import torch
    wl = W.make_custom(200, 1024, 768, 24, [8, 16, 16, 32], scale=0.7, index="zipf", tile_m=8,
                       weight_mode="unitB", frac_none=0.05, seed=77)
    wl.targets = wl.targets * 3
    wl.calls = [0, 1, 2]
    with _session(wl) as s:
        s.build_segments()
        outs = []
        for c in range(3):
            x_h, yb_h = wl.activations(c)
            x, yb = bf16_tensor(x_h, s.device), bf16_tensor(yb_h, s.device)
            y = torch.empty_like(yb)
            outs.append((x, yb, y))
        for rep in range(2):            # second round: every launch is of the early kind
            for c, (x, yb, y) in enumerate(outs):
                lb.bgmv_apply(s.pool, c, x, x.shape[1], yb, yb.shape[1], y, y.shape[1], s.slot_idx_dev,
                              wl.T, s.meta, s.ws, stream=s.compute)
        torch.cuda.synchronize()
        for c, (x, yb, y) in enumerate(outs):
            y_ref, _ = oracle_full(wl, call=c)
            check_tolerance(_bits(y), y_ref, what="apply %d of 3 on one table" % c)
        assert s.status()[1] == 0


def test_graph_replay_of_rotating_steps_matches_oracle():
    """The launch configuration bench.py times: a CUDA graph of consecutive steps (metadata build +
    grouped apply) over rotating copies of the config-1 projection, replayed several times.  Every
    copy's result is compared with the oracle, and a replay must reproduce the first one bit for bit."""
    import torch
    from paper_2602_24044_b200 import binding as lb
    from paper_2602_24044_b200.harness import bf16_tensor
    wl = W.make_config(1)
    R = 3
    wl.targets = wl.targets * R
    wl.calls = list(range(R))
    with _session(wl, a_layout=lb.A_RANK_MAJOR) as s:
        T = wl.T
        nwords = lb.segments_bytes(T, wl.num_slots, wl.tile_m) // 4
        sets, metas = [], []
        for r in range(R):
            x_h, yb_h = wl.activations(r)
            x, yb = bf16_tensor(x_h, s.device), bf16_tensor(yb_h, s.device)
            sets.append((x, yb, torch.empty_like(yb)))
            metas.append(torch.empty(nwords, dtype=torch.int32, device=s.device))

        def step(r):
            x, yb, y = sets[r]
            lb.build_segments(s.pool, s.slot_idx_dev, T, wl.tile_m, wl.long_min, metas[r], stream=s.compute)
            lb.bgmv_apply(s.pool, r, x, x.shape[1], yb, yb.shape[1], y, y.shape[1], s.slot_idx_dev, T,
                          metas[r], s.ws, stream=s.compute)

        with torch.cuda.stream(s.compute):
            for r in range(R):
                step(r)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=s.compute):
            for r in range(R):
                step(r)
        with torch.cuda.stream(s.compute):
            g.replay()
        first = [_bits(sets[r][2]).copy() for r in range(R)]
        for r in range(R):
            sets[r][2].zero_()
        with torch.cuda.stream(s.compute):
            for _ in range(3):
                g.replay()
        for r in range(R):
            y_ref, _ = oracle_full(wl, call=r)
            got = _bits(sets[r][2])
            check_tolerance(got, y_ref, what="graph replay, copy %d" % r)
            assert np.array_equal(got, first[r])
        assert s.status()[1] == 0

def test_two_layer_step_in_a_graph_with_swap_in_on_the_side_stream():
    """Config 4 cut to two layers, run the way bench.py runs the 32-layer step: one metadata build
    and 14 applies captured in a CUDA graph and replayed, while adapters that the step's tokens do
    not use are swapped into their slots on the load stream.  All 14 outputs against the oracle."""
    import torch
    from paper_2602_24044_b200 import binding as lb
    from paper_2602_24044_b200.harness import bf16_tensor
    wl = W.make_config(4, layers=2)
    n_calls = len(wl.calls)
    with _session(wl, a_layout=lb.A_RANK_MAJOR) as s:
        T = wl.T
        meta = torch.empty(lb.segments_bytes(T, wl.num_slots, wl.tile_m) // 4, dtype=torch.int32,
                           device=s.device)
        bufs = []
        for c in range(n_calls):
            x_h, yb_h = wl.activations(c)
            x, yb = bf16_tensor(x_h, s.device), bf16_tensor(yb_h, s.device)
            bufs.append((x, yb, torch.empty_like(yb)))

        def step():
            lb.build_segments(s.pool, s.slot_idx_dev, T, wl.tile_m, wl.long_min, meta, stream=s.compute)
            for c, (x, yb, y) in enumerate(bufs):
                lb.bgmv_apply(s.pool, s.target_pos[wl.calls[c]], x, x.shape[1], yb, yb.shape[1], y,
                              y.shape[1], s.slot_idx_dev, T, meta, s.ws, stream=s.compute)

        with torch.cuda.stream(s.compute):
            step()
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=s.compute):
            step()
        for _, _, y in bufs:
            y.zero_()
        victims = [int(v) for v in wl.swap_victims[:4]]
        used = set(int(v) for v in wl.distinct_slots())
        assert not used & set(victims)
        blobs = [s.host_adapter_packed(v) for v in victims]
        with torch.cuda.stream(s.compute):
            g.replay()
            for v, (A, B) in zip(victims, blobs):       # the same adapters again: contents unchanged
                lb.pool_load_slot(s.pool, v, int(wl.ranks[v]), float(wl.scales[v]), A, B, lb.PACKED,
                                  s.load, None, False)
            g.replay()
        torch.cuda.synchronize()
        for c, (x, yb, y) in enumerate(bufs):
            y_ref, _ = oracle_full(wl, c)
            check_tolerance(_bits(y), y_ref, what="two-layer step, projection %d" % c)
        assert s.status()[1] == 0
