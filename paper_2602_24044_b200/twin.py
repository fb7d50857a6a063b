"""A digital twin of one LLM-adapter serving GPU: the continuous-batching loop of the paper
(Section 5, Fig. 3) as a CPU program, driven by the four estimators of Section 5.2, Eq. 1.

Each step: requests that have arrived join the pending queue; the scheduler drops finished
requests and admits pending ones in arrival order while their tokens fit into T_max
(= Mem_max(A_max, S_max)) and the batch names at most A_max distinct adapters (greedy KV
allocation: a request is charged its prompt plus the tokens it has produced so far); the adapter
cache loads the adapters of the batch that are not resident (least recently used ones make room;
bookkeeping by the library's slot policy, lora_policy_admit); the model advances every running
request by one token.  Simulated time advances by Lat_sched + sum Lat_load + Lat_model per step.

The estimators' constants are inputs.  ``Estimators.from_sweep`` takes the adapter terms from
this library's own measurements (``bench.py --sweep``: Overhead_A as microseconds per layer
projection, Lat_load as milliseconds per adapter size); the backbone and scheduler constants have
no counterpart in this library and keep caller-given (or default, illustrative) values.

Outputs: throughput (input + output tokens per second, the paper's definition in Section 8.1),
mean inter-token latency, mean time to first token, the share of offered tokens served (the
starvation criterion of Section 6: below 90 % counts as starving).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence

import numpy as np

from . import binding as lb


@dataclass
class Request:
    arrival: float        # seconds
    adapter: int          # adapter id (-1: backbone only)
    size: int             # adapter rank
    n_in: int             # prompt tokens
    n_out: int            # output tokens to produce (given to the twin, Section 5)


@dataclass
class Estimators:
    """Eq. 1.  Times in seconds."""
    k1: float = 2.0e-6     # Lat_sched = k1 * B + k2 * R_P + k3 * R_P * A_B / A
    k2: float = 1.0e-6
    k3: float = 5.0e-6
    k4: float = 4.0e-5     # Lat_backbone = k4 * B + k5
    k5: float = 8.0e-3
    k6: float = 1.0e-3     # Overhead_A = k6 * A_B + k7   (dimensionless factor on the backbone latency)
    k7: float = 1.0
    load_ms_per_mb: float = 0.0172   # Lat_load(S) = a * S[MB] + b
    load_ms_const: float = 0.39
    mb_per_rank: float = 5.24        # adapter megabytes per unit of rank (Llama-3-8B shapes, bf16)
    t_max_base: int = 200_000        # Mem_max: tokens that fit with no adapter slot reserved
    tokens_per_slot_rank: float = 2.6   # tokens of KV cache one slot of rank 1 displaces

    def lat_sched(self, B: int, r_pending: int, a_batch: int, a_total: int) -> float:
        return self.k1 * B + self.k2 * r_pending + self.k3 * r_pending * (a_batch / max(a_total, 1))

    def lat_load(self, size: int) -> float:
        return 1e-3 * (self.load_ms_per_mb * self.mb_per_rank * size + self.load_ms_const)

    def lat_model(self, B: int, a_batch: int) -> float:
        return (self.k4 * B + self.k5) * (self.k6 * a_batch + self.k7)

    def mem_max(self, a_max: int, s_max: int) -> int:
        return max(0, int(self.t_max_base - self.tokens_per_slot_rank * a_max * s_max))

    @classmethod
    def from_sweep(cls, sweep: dict, rank: int = 16, applies_per_step: int = 224, **kw) -> "Estimators":
        """Adapter terms from a ``bench.py --sweep`` result: the fitted per-apply overhead
        (K6, K7 in microseconds at the given rank) times the adapted projections of a step, turned
        into the multiplicative form of Eq. 1 against the backbone's constant term; Lat_load from
        the fitted line."""
        e = cls(**kw)
        fit = [f for f in sweep["fits"] if f.get("rank") == rank][0]
        add_per_adapter = fit["K6_us_per_adapter"] * 1e-6 * applies_per_step
        add_const = fit["K7_us"] * 1e-6 * applies_per_step
        e.k6 = add_per_adapter / e.k5
        e.k7 = 1.0 + add_const / e.k5
        ld = [f for f in sweep["fits"] if "a_ms_per_MB" in f][0]
        e.load_ms_per_mb, e.load_ms_const = ld["a_ms_per_MB"], ld["b_ms"]
        return e


@dataclass
class TwinResult:
    throughput: float          # (input + output tokens) / duration
    itl: float                 # mean seconds between output tokens of a request
    ttft: float                # mean seconds from arrival to first output token
    served_share: float        # tokens processed / tokens offered within the duration
    steps: int
    loads: int
    finished: int
    mean_batch: float
    tokens: int = 0            # input + output tokens processed
    seconds: float = 0.0       # simulated time the throughput refers to

    @property
    def starved(self) -> bool:
        return self.served_share < 0.9


@dataclass
class _Running:
    req: Request
    produced: int = 0
    first_token_at: Optional[float] = None
    last_token_at: Optional[float] = None
    gaps: List[float] = field(default_factory=list)


def simulate(requests: Sequence[Request], a_max: int, duration: float, est: Estimators,
             n_adapters: Optional[int] = None, s_max: Optional[int] = None,
             max_steps: int = 2_000_000) -> TwinResult:
    """Run the loop for `duration` simulated seconds over requests sorted by arrival."""
    reqs = sorted(requests, key=lambda r: r.arrival)
    if s_max is None:
        s_max = max([r.size for r in reqs if r.adapter >= 0] or [0])
    if n_adapters is None:
        n_adapters = len({r.adapter for r in reqs if r.adapter >= 0})
    t_max = est.mem_max(a_max, s_max)
    policy = lb.policy_create(max(a_max, 1))
    try:
        now, nxt = 0.0, 0
        pending: List[Request] = []
        running: List[_Running] = []
        done: List[_Running] = []
        tokens_done = 0
        steps = loads = 0
        batch_sum = 0
        while now < duration and steps < max_steps:
            while nxt < len(reqs) and reqs[nxt].arrival <= now:
                pending.append(reqs[nxt])
                nxt += 1
            # scheduler: finished requests leave, pending ones are admitted in order
            still = []
            for r in running:
                (done if r.produced >= r.req.n_out else still).append(r)
            running = still
            used = sum(r.req.n_in + r.produced for r in running)
            names = {r.req.adapter for r in running if r.req.adapter >= 0}
            while pending:
                q = pending[0]
                new_names = names | ({q.adapter} if q.adapter >= 0 else set())
                if used + q.n_in > t_max or len(new_names) > a_max:
                    break
                pending.pop(0)
                running.append(_Running(q))
                used += q.n_in
                names = new_names
            if not running:
                # idle: jump to the next arrival
                if nxt >= len(reqs):
                    break
                now = max(now, reqs[nxt].arrival)
                continue
            step_time = est.lat_sched(len(running), len(pending), len(names), n_adapters)
            # adapter cache: what the batch needs and is not resident is loaded
            ids = [r.req.adapter for r in running]
            size_of: Dict[int, int] = {r.req.adapter: r.req.size for r in running}
            _, misses = lb.policy_admit(policy, ids)
            for _, adapter in misses:
                step_time += est.lat_load(size_of[adapter])
            loads += len(misses)
            # model: one token for every running request (the first step of a request is its prefill)
            step_time += est.lat_model(len(running), len(names))
            now += step_time
            for r in running:
                if r.first_token_at is None:
                    r.first_token_at = now
                    tokens_done += r.req.n_in
                else:
                    r.gaps.append(now - r.last_token_at)
                r.last_token_at = now
                r.produced += 1
                tokens_done += 1
            batch_sum += len(running)
            steps += 1
        elapsed = max(now, 1e-9)
        horizon = min(duration, elapsed) if nxt >= len(reqs) and not running and not pending else duration
        offered = sum(r.n_in + r.n_out for r in reqs if r.arrival <= horizon)
        everyone = done + running
        gaps = [g for r in everyone for g in r.gaps]
        firsts = [r.first_token_at - r.req.arrival for r in everyone if r.first_token_at is not None]
        return TwinResult(throughput=tokens_done / max(horizon, 1e-9),
                          itl=float(np.mean(gaps)) if gaps else 0.0,
                          ttft=float(np.mean(firsts)) if firsts else 0.0,
                          served_share=tokens_done / offered if offered else 1.0,
                          steps=steps, loads=loads,
                          finished=len(done) + sum(1 for r in running if r.produced >= r.req.n_out),
                          mean_batch=batch_sum / steps if steps else 0.0, tokens=tokens_done,
                          seconds=horizon)
    finally:
        lb.policy_destroy(policy)


def poisson_workload(adapters, duration: float, n_in: int = 250, n_out: int = 231, seed: int = 0) -> List[Request]:
    """Requests of `adapters` (objects with name, size, rate) with Poisson arrivals over `duration`
    seconds and the mean lengths the paper's Fig. 1 uses (250 in, 231 out)."""
    rng = np.random.default_rng(seed)
    out: List[Request] = []
    for a in adapters:
        if a.rate <= 0:
            continue
        n = rng.poisson(a.rate * duration)
        for t in np.sort(rng.uniform(0.0, duration, n)):
            out.append(Request(float(t), a.name, a.size, n_in, n_out))
    out.sort(key=lambda r: r.arrival)
    return out


def twin_predictors(est: Estimators, duration: float = 120.0, seed: int = 0):
    """The two predictors the placement algorithm asks for, answered by running the twin itself
    (the paper distils ML models from such runs; calling the twin directly is the slow, exact form)."""
    cache: Dict[tuple, TwinResult] = {}

    def run(adapters, a_max: int) -> TwinResult:
        key = (tuple(sorted((a.name, a.size, a.rate) for a in adapters)), a_max)
        if key not in cache:
            reqs = poisson_workload(adapters, duration, seed=seed)
            cache[key] = simulate(reqs, a_max, duration, est, n_adapters=len(adapters),
                                  s_max=max([a.size for a in adapters] or [0]))
        return cache[key]

    return (lambda adapters, a_max: run(adapters, a_max).throughput,
            lambda adapters, a_max: run(adapters, a_max).starved)
