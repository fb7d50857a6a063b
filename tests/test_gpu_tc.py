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
