"""GPU parity of the tensor-core (tcgen05 + TMA) path that lora_sgmv_apply uses for full tiles of
128 consecutive tokens, against the fp64 oracle and against the fused kernel."""
import numpy as np
import pytest

from gpu_util import check_tolerance, oracle_full, require_gpu
from paper_2602_24044_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _gpu():
    require_gpu()


def _run(wl, tuning=None, **kw):
    from paper_2602_24044_b200 import binding as lb
    from paper_2602_24044_b200.harness import Session, bf16_bits
    if tuning is None:
        tuning = {4: 2}   # these batches are short: force the tensor-core kernels wherever they apply
    with Session(wl, tuning=tuning) as s:
        before = lb.launch_count()
        y = bf16_bits(s.apply(**kw))
        launches = lb.launch_count() - before
        assert s.status()[1] == 0          # no bounded wait expired
    return y, launches


@pytest.mark.parametrize("ranks", [[16], [8, 16, 32, 64], [1, 24, 40]])
def test_long_sorted_segments(ranks):
    wl = W.make_custom(1000, 1024, 1536, 5, ranks, kind="sgmv", index="sorted", tile_m=128,
                       scale=[0.6, 1.3], weight_mode="unitB", seed=51)
    y_ref, _ = oracle_full(wl)
    y, n_tc = _run(wl)
    check_tolerance(y, y_ref, what="tensor-core path")
    y_f, n_fused = _run(wl, tuning={4: 1})
    check_tolerance(y_f, y_ref, what="fused only")
    assert n_tc > n_fused                      # the tensor-core kernels really ran


def test_ragged_widths_and_in_place():
    """d_in and d_out that are not multiples of the 64-column TMA box; result written in place."""
    wl = W.make_custom(700, 2312, 1544, 4, [8, 32], kind="sgmv", index="sorted", tile_m=128,
                       scale=0.8, weight_mode="unitB", frac_none=0.05, seed=52)
    y_ref, _ = oracle_full(wl)
    y, _ = _run(wl, in_place=True)
    check_tolerance(y, y_ref, what="ragged widths, in place")


def test_exact_integers_bit_exact_on_tensor_cores():
    wl = W.make_custom(640, 2048, 1024, 3, [4, 16, 32], kind="sgmv", index="sorted", tile_m=128,
                       scale=2.0, weight_mode="int", act_mode="int", seed=53)
    y_ref, _ = oracle_full(wl)
    assert np.abs(y_ref).max() < 256
    y, _ = _run(wl)
    assert np.array_equal(W.bf16_to_f64(y), y_ref)


def test_mixed_batch_scattered_and_long_tiles():
    """Decode tokens scattered over many adapters followed by whole chunks of one adapter each:
    the long chunks take the tensor-core path, everything else the fused kernel."""
    rng = np.random.default_rng(54)
    dec = rng.integers(0, 12, 150)
    slot_idx = np.concatenate([dec, np.repeat([3, 7], 256)]).astype(np.int32)
    wl = W.make_custom(0, 1024, 768, 12, [8, 16, 32, 64], kind="sgmv", tile_m=128, scale=1.1,
                       weight_mode="unitB", slot_idx=slot_idx, seed=54)
    y_ref, _ = oracle_full(wl)
    y, _ = _run(wl)
    check_tolerance(y, y_ref, what="mixed batch")


@pytest.mark.parametrize("slabs", [1, 2, 3, 5, 8])
def test_workspace_that_holds_few_partial_slabs(slabs):
    """The shrink cuts every tile's K range into pieces, one fp32 slab of the workspace per piece;
    a smaller workspace means fewer, longer pieces (one slab: whole tiles only).  Same result."""
    wl = W.make_custom(1000, 1024, 1536, 5, [8, 16, 32], kind="sgmv", index="sorted", tile_m=128,
                       scale=[0.6, 1.3], weight_mode="unitB", seed=56)
    y_ref, _ = oracle_full(wl)
    per_slab = wl.T * 32 * 4            # tokens x rank bucket of the pool x fp32
    y, n = _run(wl, ws_bytes=slabs * per_slab + 4096)   # the work list fits in the slack
    check_tolerance(y, y_ref, what="%d slabs" % slabs)
    _, n_fused = _run(wl, tuning={4: 1})
    assert n > n_fused                  # the tensor-core kernels took their tiles


def test_prefill_apply_in_a_cuda_graph():
    """lora_sgmv_apply forks the leftover tiles onto the pool's own stream and joins it back; the
    whole call must be capturable and a replay must reproduce the eager result bit for bit."""
    import torch
    from paper_2602_24044_b200 import binding as lb
    from paper_2602_24044_b200.harness import Session, bf16_bits, bf16_tensor
    rng = np.random.default_rng(57)
    dec = rng.integers(0, 12, 90)
    slot_idx = np.concatenate([np.repeat([2, 5], 300), dec, np.repeat([9], 200)]).astype(np.int32)
    wl = W.make_custom(0, 1024, 768, 12, [8, 16, 32], kind="sgmv", tile_m=128, scale=0.9,
                       weight_mode="unitB", slot_idx=slot_idx, seed=57)
    y_ref, _ = oracle_full(wl)
    with Session(wl, tuning={4: 2}) as s:
        x_h, yb_h = wl.activations(0)
        x, yb = bf16_tensor(x_h, s.device), bf16_tensor(yb_h, s.device)
        y = torch.empty_like(yb)
        nwords = lb.segments_bytes(wl.T, wl.num_slots, wl.tile_m) // 4
        meta = torch.empty(nwords, dtype=torch.int32, device=s.device)

        def step():
            lb.build_segments(s.pool, s.slot_idx_dev, wl.T, wl.tile_m, wl.long_min, meta, stream=s.compute)
            lb.sgmv_apply(s.pool, 0, x, x.shape[1], yb, yb.shape[1], y, y.shape[1], meta, wl.T, s.ws,
                          stream=s.compute)

        with torch.cuda.stream(s.compute):
            step()
        eager = bf16_bits(y).copy()
        check_tolerance(eager, y_ref, what="eager")
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=s.compute):
            step()
            step()
        for _ in range(3):
            y.view(torch.int16).fill_(0x7F7F)
            torch.cuda.synchronize()
            with torch.cuda.stream(s.compute):
                g.replay()
            assert np.array_equal(bf16_bits(y), eager)
        assert s.status()[1] == 0


def test_leftover_tiles_beside_or_after_the_tensor_core_kernels_give_the_same_bits():
    """The tiles the tensor-core kernels leave over run on the pool's own stream beside them
    (default) or after them on the caller's stream (tuning key 6 = 1): disjoint rows, same result."""
    rng = np.random.default_rng(58)
    dec = rng.integers(0, 10, 120)
    slot_idx = np.concatenate([np.repeat([1, 4], 260), dec, np.repeat([4], 70), np.repeat([8], 150)]).astype(np.int32)
    wl = W.make_custom(0, 1536, 1024, 10, [8, 16, 32], kind="sgmv", tile_m=128, scale=1.2,
                       weight_mode="unitB", slot_idx=slot_idx, frac_none=0.03, seed=58)
    y_ref, _ = oracle_full(wl)
    y_beside, n_beside = _run(wl)
    y_after, n_after = _run(wl, tuning={4: 2, 6: 1})
    check_tolerance(y_beside, y_ref, what="beside")
    assert np.array_equal(y_beside, y_after)
    assert n_beside == n_after
