"""The digital-twin loop (paper Section 5) and the caching greedy algorithm (Section 7, Algorithms
1 and 2) as CPU programs: hand-worked orderings, invariants of the placement, stub predictors that
force every branch (commit, rollback, starvation), conservation and limiting cases of the twin."""
import numpy as np
import pytest

from conftest import read_golden
from paper_2602_24044_b200 import build as lbuild
from paper_2602_24044_b200 import placement as pl
from paper_2602_24044_b200 import twin as tw


@pytest.fixture(scope="module", autouse=True)
def _lib():
    lbuild.build()


def test_priority_sorting_hand_example():
    g = read_golden("priority_sorting_hand.txt")
    ads = [pl.Adapter(i, int(s), r) for i, (s, r) in enumerate(zip(g["sizes"], g["rates"]))]
    assert [a.name for a in pl.priority_sorting(ads)] == [int(v) for v in g["order"]]


def test_next_config_walks_the_testing_points():
    assert [pl.next_gpu_config(p) for p in (0, 8, 9, 64, 320, 384, 500)] == [8, 16, 16, 96, 384, 384, 384]


def _capacity_predictors(cap):
    """A GPU serves up to `cap` adapters at full rate and starves beyond; a larger A_max than
    needed costs throughput (memory taken from the KV cache), so the smallest fitting one wins."""
    def thr(ads, p):
        return sum(a.rate for a in ads[:min(len(ads), p)]) * 481.0 - 0.01 * p
    def starve(ads, p):
        return len(ads) > cap or p < min(len(ads), cap)
    return thr, starve


def test_greedy_packs_first_fit_and_configures_amax():
    rng = np.random.default_rng(3)
    ads = [pl.Adapter(i, int(rng.choice([8, 16, 32])), float(rng.choice([0.1, 0.4, 1.6]))) for i in range(100)]
    thr, starve = _capacity_predictors(40)
    assign, a_max = pl.greedy_caching(ads, 4, thr, starve)
    assert sorted(assign) == list(range(100))                 # every adapter placed exactly once
    per_gpu = [sum(1 for g in assign.values() if g == i) for i in range(4)]
    # testing points 8, 16, 32 pass on a GPU, 64 fails and rolls 32 adapters back to the next GPU;
    # the last GPU in use keeps 36 (never reaches 64; tested at the end, where 64 slots serve more
    # of its 36 adapters than 32 do)
    assert per_gpu == [32, 32, 36, 0]
    assert a_max == [32, 32, 64, 0]
    # the largest adapters were placed first: GPU 0 holds only the largest sizes present
    order = pl.priority_sorting(ads)
    assert {a.name for a in order[:32]} == {n for n, g in assign.items() if g == 0}


def test_greedy_raises_when_gpus_run_out_and_when_the_tail_starves():
    ads = [pl.Adapter(i, 16, 0.4) for i in range(70)]
    thr, starve = _capacity_predictors(24)       # 16 per GPU pass the test, 32 do not
    with pytest.raises(pl.Starvation):
        pl.greedy_caching(ads, 3, thr, starve)   # three GPUs keep 16 each, 22 adapters are left over
    assign, a_max = pl.greedy_caching(ads, 4, thr, starve)
    # the fourth GPU keeps its 16 and the 6 that are left: 22 never reaches the testing point 32
    assert [sum(1 for g in assign.values() if g == i) for i in range(4)] == [16, 16, 16, 22]
    # with room for 20 only, those 22 fail the closing test: the algorithm does not retry there
    with pytest.raises(pl.Starvation):
        pl.greedy_caching(ads, 5, *_capacity_predictors(20))
    # a tail that is never tested inside the loop is tested at the end
    with pytest.raises(pl.Starvation):
        pl.greedy_caching([pl.Adapter(i, 8, 1.0) for i in range(5)], 1, thr, lambda a, p: True)


def test_test_allocation_prefers_the_better_configuration():
    g = pl.GpuState(0, allocated=[pl.Adapter(i, 8, 0.1) for i in range(8)], a_max=8,
                    provisional=[pl.Adapter(8 + i, 8, 0.1) for i in range(8)])
    ok, alloc, p = pl.test_allocation(g, lambda a, p: float(p), lambda a, p: False)
    assert ok and p == 16 and [a.name for a in alloc] == list(range(8, 16))
    ok, alloc, p = pl.test_allocation(g, lambda a, p: -float(p), lambda a, p: False)
    assert ok and p == 8
    assert pl.test_allocation(g, lambda a, p: 1.0, lambda a, p: True) == (False, [], 0)


# ---------------------------------------------------------------------------------------------
# the twin
# ---------------------------------------------------------------------------------------------
def test_twin_serves_a_light_load_completely():
    est = tw.Estimators()
    ads = [pl.Adapter(i, 16, 0.2) for i in range(8)]
    reqs = tw.poisson_workload(ads, 200.0, seed=1)
    res = tw.simulate(reqs, a_max=8, duration=400.0, est=est)
    assert res.finished == len(reqs) and not res.starved
    offered = sum(r.n_in + r.n_out for r in reqs)
    assert res.tokens == offered                                            # every token counted once
    assert res.throughput == pytest.approx(offered / res.seconds)
    assert res.loads == 8                                                   # each adapter loaded once: all fit
    # an isolated request: first token after one step, then one token per step
    one = tw.simulate([tw.Request(0.0, 0, 16, 100, 10)], 8, 10.0, est)
    step = est.lat_sched(1, 0, 1, 1) + est.lat_model(1, 1)
    assert one.ttft == pytest.approx(step + est.lat_load(16)) and one.itl == pytest.approx(step)
    assert one.steps == 10 and one.loads == 1


def test_twin_swaps_when_amax_is_smaller_than_the_working_set():
    est = tw.Estimators()
    # two adapters, strictly alternating requests that never overlap, one slot: every request loads
    reqs = [tw.Request(2.0 * i, i % 2, 32, 50, 5) for i in range(20)]
    res = tw.simulate(reqs, a_max=1, duration=100.0, est=est)
    assert res.loads == 20 and res.finished == 20
    res2 = tw.simulate(reqs, a_max=2, duration=100.0, est=est)
    assert res2.loads == 2 and res2.ttft < res.ttft


def test_twin_starves_under_overload_and_amax_trades_memory_for_adapters():
    est = tw.Estimators(t_max_base=6000, tokens_per_slot_rank=10.0)
    ads = [pl.Adapter(i, 16, 3.0) for i in range(16)]
    reqs = tw.poisson_workload(ads, 60.0, seed=2)
    small = tw.simulate(reqs, a_max=2, duration=60.0, est=est)
    assert small.starved and small.served_share < 0.9
    # more slots admit more adapters per batch, until the slots have eaten the KV cache
    mid = tw.simulate(reqs, a_max=8, duration=60.0, est=est)
    huge = tw.simulate(reqs, a_max=36, duration=60.0, est=est)   # T_max = 6000 - 10*36*16 = 240 < one prompt
    assert mid.throughput > small.throughput and huge.throughput == 0.0
    # determinism
    assert tw.simulate(reqs, 8, 60.0, est) == mid


def test_estimators_from_a_sweep_and_twin_predictors_in_the_greedy_algorithm():
    sweep = {"fits": [{"rank": 16, "K6_us_per_adapter": 0.05, "K7_us": 7.5},
                      {"model": "Lat_load", "a_ms_per_MB": 0.017, "b_ms": 0.4}]}
    est = tw.Estimators.from_sweep(sweep, rank=16, applies_per_step=224)
    assert est.k7 == pytest.approx(1.0 + 7.5e-6 * 224 / est.k5)
    assert est.lat_model(32, 10) > est.lat_model(32, 1) > tw.Estimators(k6=0.0, k7=1.0).lat_model(32, 1)
    assert est.lat_load(64) == pytest.approx(1e-3 * (0.017 * est.mb_per_rank * 64 + 0.4))
    thr, starve = tw.twin_predictors(est, duration=30.0)
    ads = [pl.Adapter(i, 8, 0.05) for i in range(24)]
    assign, a_max = pl.greedy_caching(ads, 2, thr, starve)
    assert sorted(assign) == list(range(24)) and set(assign.values()) == {0}   # a light load fits one GPU
    assert a_max[0] in pl.TESTING_POINTS and a_max[1] == 0
