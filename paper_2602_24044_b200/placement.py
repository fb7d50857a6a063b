"""Adapter placement: the caching greedy algorithm of the paper (Section 7, Algorithms 1 and 2) as a
CPU program with pluggable predictors.

Given the adapters to serve (expected size and Poisson arrival rate each) and the GPUs of a node,
decide which GPU hosts which adapter and how many adapter slots (A_max) each GPU's pool gets,
using as few GPUs as possible while no GPU starves.  The paper drives the algorithm with ML models
distilled from its Digital Twin; here the two predictors are arguments (callables), so the
algorithm runs with the twin itself (``twin.twin_predictors``), with a fitted model, or with a
stub in tests.

Readings of the paper where it leaves room (Section 7 omits "internal state management"):
  * PrioritySorting: sizes descending; inside one size the rates alternate highest, lowest,
    second highest, second lowest, ... (the "zigzag" of the text).
  * The GPU queue: the GPU at the head takes adapters until a test fails on it; a failed test
    rolls its provisional adapters back into the pending queue (in front, in their order) and the
    GPU leaves the queue with what it had committed, so the next GPU takes over.
  * ReachTestingPoint: the number of adapters on the GPU (committed + provisional) equals one of
    the testing points [8, 16, 32, 64, 96, 128, 160, 192, 256, 320, 384].
  * NextGPUConfig: the smallest testing point above the GPU's current A_max, or the largest one.
    A GPU that has no configuration yet (A_max = 0) is tested at the first two points.
"""
from __future__ import annotations

from collections import deque
from dataclasses import dataclass, field
from typing import Callable, Dict, List, Sequence, Tuple

TESTING_POINTS = [8, 16, 32, 64, 96, 128, 160, 192, 256, 320, 384]


class Starvation(RuntimeError):
    """No starvation-free allocation exists with the GPUs given (Algorithm 1's error)."""


@dataclass(frozen=True)
class Adapter:
    name: int
    size: int        # LoRA rank (the adapter "size" of the paper)
    rate: float      # requests per second (Poisson)


# predictors: (adapters on the GPU, A_max) -> tokens/s  /  -> True when the GPU would starve
ThroughputFn = Callable[[Sequence[Adapter], int], float]
StarvationFn = Callable[[Sequence[Adapter], int], bool]


def priority_sorting(adapters: Sequence[Adapter]) -> List[Adapter]:
    """Largest size first; inside a size, rates in zigzag order (high, low, next high, ...)."""
    out: List[Adapter] = []
    for size in sorted({a.size for a in adapters}, reverse=True):
        group = sorted((a for a in adapters if a.size == size), key=lambda a: (-a.rate, a.name))
        lo, hi = 0, len(group) - 1
        take_high = True
        while lo <= hi:
            if take_high:
                out.append(group[lo])
                lo += 1
            else:
                out.append(group[hi])
                hi -= 1
            take_high = not take_high
    return out


def next_gpu_config(p: int) -> int:
    """The next candidate A_max after p among the testing points (the last one stays)."""
    for t in TESTING_POINTS:
        if t > p:
            return t
    return TESTING_POINTS[-1]


@dataclass
class GpuState:
    index: int
    allocated: List[Adapter] = field(default_factory=list)     # committed
    provisional: List[Adapter] = field(default_factory=list)   # included, not yet tested
    a_max: int = 0

    def count(self) -> int:
        return len(self.allocated) + len(self.provisional)


def test_allocation(gpu: GpuState, predict_throughput: ThroughputFn,
                    predict_starvation: StarvationFn) -> Tuple[bool, List[Adapter], int]:
    """Algorithm 2: throughput at the current and at the next A_max, the better one is kept; the
    allocation is feasible if the GPU does not starve with it."""
    p = gpu.a_max if gpu.a_max > 0 else TESTING_POINTS[0]
    p_next = next_gpu_config(p)
    everything = gpu.allocated + gpu.provisional
    t = predict_throughput(everything, p)
    t_next = predict_throughput(everything, p_next)
    p_best = p if t > t_next else p_next
    if predict_starvation(everything, p_best):
        return False, [], 0
    return True, list(gpu.provisional), p_best


def greedy_caching(adapters: Sequence[Adapter], n_gpus: int, predict_throughput: ThroughputFn,
                   predict_starvation: StarvationFn):
    """Algorithm 1.  Returns (assignment {adapter name: gpu index}, a_max per gpu [n_gpus]).
    Raises Starvation when the adapters cannot be placed without a starving GPU."""
    gpus = [GpuState(i) for i in range(n_gpus)]
    assignment: Dict[int, int] = {}
    pending = deque(priority_sorting(adapters))
    gpu_q = deque(gpus)

    def commit(g: GpuState, alloc: List[Adapter], p_new: int) -> None:
        g.allocated += alloc
        g.provisional = []
        for a in alloc:
            assignment[a.name] = g.index
        g.a_max = p_new

    while pending:
        a = pending.popleft()
        if not gpu_q:
            raise Starvation("adapter %d and %d more cannot be placed" % (a.name, len(pending)))
        g = gpu_q.popleft()
        g.provisional.append(a)
        if g.count() in TESTING_POINTS:
            ok, alloc, p_new = test_allocation(g, predict_throughput, predict_starvation)
            if ok:
                commit(g, alloc, p_new)
                gpu_q.appendleft(g)
            else:
                # roll back: the provisional adapters return to the head of the queue in their
                # order; this GPU keeps what it had committed and takes no more
                for b in reversed(g.provisional):
                    pending.appendleft(b)
                g.provisional = []
        else:
            gpu_q.appendleft(g)
    for g in gpus:
        if g.provisional:
            ok, alloc, p_new = test_allocation(g, predict_throughput, predict_starvation)
            if not ok:
                raise Starvation("GPU %d starves with its last %d adapters" % (g.index, len(g.provisional)))
            commit(g, alloc, p_new)
    return assignment, [g.a_max for g in gpus]
