"""Host-side slot policy and pool sizing: checked against a brute-force model written out here
(a list scan for the least recently used slot), on random request streams and on the edge cases
(all slots pinned, more distinct adapters than slots, repeated adapters inside a batch)."""
import numpy as np
import pytest

from paper_2602_24044_b200 import binding as lb
from paper_2602_24044_b200 import build as lbuild


@pytest.fixture(scope="module", autouse=True)
def _lib():
    lbuild.build()


class Model:
    """The policy's definition, the slow way."""

    def __init__(self, n):
        self.adapter = [-1] * n
        self.stamp = [0] * n
        self.pins = [0] * n
        self.clock = 0

    def victim(self, skip=()):
        best = -1
        for s in range(len(self.adapter)):
            if self.pins[s] or s in skip:
                continue
            if self.adapter[s] < 0:
                return s
            if best < 0 or self.stamp[s] < self.stamp[best]:
                best = s
        return best

    def admit(self, batch):
        used = {self.adapter.index(a) for a in batch if a >= 0 and a in self.adapter}
        missing = []
        for a in batch:
            if a >= 0 and a not in self.adapter and a not in missing:
                missing.append(a)
        skip, victims = set(used), []
        for _ in missing:
            v = self.victim(skip)
            if v < 0:
                return None
            skip.add(v)
            victims.append(v)
        for a, v in zip(missing, victims):
            self.adapter[v] = a
        out = []
        for a in batch:
            if a < 0:
                out.append(-1)
                continue
            s = self.adapter.index(a)
            self.clock += 1
            self.stamp[s] = self.clock
            out.append(s)
        return out, list(zip(victims, missing))


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_admit_matches_the_brute_force_model(seed):
    rng = np.random.default_rng(seed)
    N = 12
    pol, ref = lb.policy_create(N), Model(N)
    pinned = []
    for step in range(300):
        batch = [int(a) for a in rng.integers(-1, 40, rng.integers(0, 10))]
        want = ref.admit(batch)
        if want is None:
            with pytest.raises(lb.LoraError) as e:
                lb.policy_admit(pol, batch)
            assert e.value.status == 6
        else:
            sidx, misses = lb.policy_admit(pol, batch)
            assert sidx.tolist() == want[0] and misses == want[1]
            for s, a in misses:
                assert lb.policy_lookup(pol, a) == s
        # pin / unpin some resident slots now and then
        if step % 7 == 0:
            res = [s for s in range(N) if ref.adapter[s] >= 0]
            pick = [int(s) for s in rng.choice(res, size=min(len(res), 9), replace=False)] if res else []
            lb.policy_pin(pol, pick)
            for s in pick:
                ref.pins[s] += 1
            pinned.append(pick)
        if step % 11 == 5 and pinned:
            pick = pinned.pop(0)
            lb.policy_unpin(pol, pick)
            for s in pick:
                ref.pins[s] -= 1
        for s in range(N):
            assert lb.policy_slot(pol, s) == (ref.adapter[s], ref.pins[s])
    lb.policy_destroy(pol)


def test_victim_order_pins_and_errors():
    pol = lb.policy_create(3)
    assert lb.policy_choose_victim(pol) == (0, -1)          # empty slots first, lowest index
    for slot, a in enumerate([100, 200, 300]):
        lb.policy_assign(pol, slot, a)
    assert lb.policy_choose_victim(pol) == (0, 100)          # oldest use
    lb.policy_touch(pol, 0)
    assert lb.policy_choose_victim(pol) == (1, 200)
    lb.policy_pin(pol, [1, 1])
    assert lb.policy_choose_victim(pol) == (2, 300)
    lb.policy_pin(pol, [0, 2])
    for call, status in [(lambda: lb.policy_choose_victim(pol), 6),
                         (lambda: lb.policy_assign(pol, 1, 999), 6),
                         (lambda: lb.policy_release(pol, 2), 6),
                         (lambda: lb.policy_admit(pol, [555]), 6),
                         (lambda: lb.policy_touch(pol, 3), 3),
                         (lambda: lb.policy_unpin(pol, [0, 0]), 1),
                         (lambda: lb.policy_assign(pol, 1, 100), 6)]:
        with pytest.raises(lb.LoraError) as e:
            call()
        assert e.value.status == status
    # a failed admit changed nothing
    assert [lb.policy_slot(pol, s) for s in range(3)] == [(100, 1), (200, 2), (300, 1)]
    lb.policy_unpin(pol, [1])
    lb.policy_unpin(pol, [1, 0, 2])
    lb.policy_release(pol, 1)
    assert lb.policy_lookup(pol, 200) == -1
    for call, status in [(lambda: lb.policy_touch(pol, 1), 5), (lambda: lb.policy_pin(pol, [1]), 5),
                         (lambda: lb.policy_release(pol, 1), 5),
                         (lambda: lb.policy_assign(pol, 1, 100), 1)]:   # 100 lives in slot 0
        with pytest.raises(lb.LoraError) as e:
            call()
        assert e.value.status == status
    # a batch naming one adapter several times loads it once; hits count distinct resident adapters
    sidx, misses = lb.policy_admit(pol, [7, 7, -1, 100, 7])
    assert misses == [(1, 7)] and sidx.tolist() == [1, 1, -1, 0, 1]
    assert lb.policy_stats(pol) == (1, 1, 0)
    # a batch with more distinct adapters than slots cannot be admitted
    with pytest.raises(lb.LoraError) as e:
        lb.policy_admit(pol, [1, 2, 3, 4])
    assert e.value.status == 6
    lb.policy_destroy(pol)


def test_pool_plan_is_the_inverse_of_pool_bytes():
    t = [(4096, 4096), (4096, 1024), (4096, 1024), (4096, 4096), (4096, 14336), (4096, 14336),
         (14336, 4096)] * 32
    n, per = lb.pool_plan(40 * 10 ** 9, t, 16)
    assert per == 83886080                                   # Llama-3-8B, rank 16, seven projections
    assert lb.pool_bytes(n, 16, t) <= 40 * 10 ** 9 < lb.pool_bytes(n + 1, 16, t)
    for budget in [lb.pool_bytes(1, 8, [(64, 64)]), lb.pool_bytes(17, 8, [(64, 64)]) + 5,
                   lb.pool_bytes(300, 8, [(64, 64)]) - 1]:
        n, _ = lb.pool_plan(budget, [(64, 64)], 8)
        assert lb.pool_bytes(n, 8, [(64, 64)]) <= budget
        assert n == 8192 or lb.pool_bytes(n + 1, 8, [(64, 64)]) > budget
    with pytest.raises(lb.LoraError) as e:
        lb.pool_plan(1000, [(64, 64)], 8)
    assert e.value.status == 7
