"""GPU parity of every kernel path and launch shape the library can be tuned to: the two-phase
kernels (tuning key 0 = 1) and the fused cluster kernel at cluster sizes 1, 2, 4, 8 (key 1)."""
import numpy as np
import pytest

from gpu_util import check_tolerance, oracle_full, require_gpu
from paper_2602_24044_b200 import workloads as W

pytestmark = pytest.mark.gpu

TUNINGS = [{0: 1}, {1: 1}, {1: 2}, {1: 4}, {1: 8}]
IDS = ["twophase", "fused-c1", "fused-c2", "fused-c4", "fused-c8"]


@pytest.fixture(scope="module", autouse=True)
def _gpu():
    require_gpu()


def _run(wl, tuning, **kw):
    from paper_2602_24044_b200.harness import Session, bf16_bits
    with Session(wl, tuning=tuning) as s:
        y = bf16_bits(s.apply(**kw))
        assert s.status()[1] == 0          # no bounded wait expired
    return y


@pytest.mark.parametrize("tuning", TUNINGS, ids=IDS)
@pytest.mark.parametrize("grouped", [True, False])
def test_decode_mixed_ranks(tuning, grouped):
    wl = W.make_custom(150, 1160, 2056, 20, [1, 5, 8, 16, 24, 32, 48, 64], scale=[0.3, 1.7],
                       index="zipf", frac_none=0.1, weight_mode="unitB", seed=41)
    y_ref, _ = oracle_full(wl)
    check_tolerance(_run(wl, tuning, grouped=grouped), y_ref, what=str(tuning))


@pytest.mark.parametrize("tuning", TUNINGS, ids=IDS)
def test_prefill_tiles_of_128_rows(tuning):
    """Long sorted segments: full 128-row tiles, ragged tails, several column chunks per block."""
    wl = W.make_custom(900, 2304, 1544, 7, [8, 16, 32, 64], kind="sgmv", index="sorted",
                       tile_m=128, scale=0.6, weight_mode="unitB", seed=42)
    y_ref, _ = oracle_full(wl)
    check_tolerance(_run(wl, tuning), y_ref, what=str(tuning))


@pytest.mark.parametrize("tuning", TUNINGS, ids=IDS)
def test_exact_integers_bit_exact(tuning):
    wl = W.make_custom(120, 2048, 1032, 9, [1, 4, 8, 16, 32], scale=2.0, weight_mode="int",
                       act_mode="int", frac_none=0.1, kind="sgmv", tile_m=64, seed=43)
    y_ref, _ = oracle_full(wl)
    assert np.abs(y_ref).max() < 256
    y = _run(wl, tuning)
    assert np.array_equal(W.bf16_to_f64(y), y_ref)


@pytest.mark.parametrize("tuning", TUNINGS[1:], ids=IDS[1:])
def test_narrow_projection_with_idle_blocks(tuning):
    """d_in and d_out so small that some blocks of a cluster own no columns."""
    wl = W.make_custom(40, 16, 24, 3, [2, 8], scale=1.5, weight_mode="unitB", seed=44)
    y_ref, _ = oracle_full(wl)
    check_tolerance(_run(wl, tuning), y_ref, what=str(tuning))
    check_tolerance(_run(wl, tuning, in_place=True), y_ref, what=str(tuning))
