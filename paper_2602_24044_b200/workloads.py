"""Seeded synthetic inputs for the multi-adapter LoRA forward.

This module only draws numbers and arranges them; it contains none of the
method's arithmetic (no products of x, A, B, no grouping of tokens).  Both the
CPU oracle's tests and the CUDA path's tests/bench take their inputs from
here, so the two sides always see the same bf16 bit patterns.

All floating-point tensors are produced as float32 draws, rounded once to
bfloat16 (round-to-nearest-even) and carried as ``numpy.uint16`` bit patterns.

Shapes and distributions follow the serving scenarios of the paper's
evaluation (hundreds of resident adapters, LoRA ranks 8/16/32, Llama-3-8B
projection sizes, ShareGPT-like prompt lengths) with synthetic stand-ins:

===  =====================================================================
cfg  workload
===  =====================================================================
0    decode, 16 tokens, 1024->1024, 8 adapters rank 8, uniform slot per token
1    decode, 256 tokens, 4096->4096, 128 adapters rank 16, Zipf(1.1) slots
2    prefill, 32 requests, lognormal lengths (median 512, sigma 1, clip
     32..2048), 4096->14336 and 14336->4096, 64 adapters, ranks {8,16,32}
3    mixed: 512 decode tokens + 4 prefill chunks of 512, 4096->6144,
     384 adapters, ranks {8,16,32,64}, Zipf(0.9)
4    32-layer step, 7 projections per layer (Llama-3-8B shapes), 256 decode
     tokens, 256 adapters rank 16, Zipf(1.1), 16 swap-in victims per step
===  =====================================================================
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

SEED_BASE = 26022404


# --------------------------------------------------------------------------
# bf16 helpers (format conversion only)
# --------------------------------------------------------------------------
def bf16_round(a: np.ndarray) -> np.ndarray:
    """float32 -> bfloat16 bit patterns (uint16), round-to-nearest-even."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_to_f32(h: np.ndarray) -> np.ndarray:
    """bfloat16 bit patterns -> float32 (exact)."""
    h = np.ascontiguousarray(h, dtype=np.uint16)
    return (h.astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_to_f64(h: np.ndarray) -> np.ndarray:
    """bfloat16 bit patterns -> float64 (exact)."""
    return bf16_to_f32(h).astype(np.float64)


# --------------------------------------------------------------------------
# distributions
# --------------------------------------------------------------------------
def bounded_zipf(rng: np.random.Generator, n_items: int, s: float, size: int) -> np.ndarray:
    """Draw ``size`` items from p(k) ~ k^-s, k = 1..n_items; returns k-1 (int32).

    Inverse-CDF sampling on float64 cumulative sums.
    """
    w = np.arange(1, n_items + 1, dtype=np.float64) ** (-float(s))
    cdf = np.cumsum(w)
    cdf /= cdf[-1]
    u = rng.random(size)
    k = np.searchsorted(cdf, u, side="right")
    return np.minimum(k, n_items - 1).astype(np.int32)


def lognormal_lengths(rng: np.random.Generator, n: int, median: float, sigma: float,
                      lo: int, hi: int) -> np.ndarray:
    z = rng.standard_normal(n)
    ln = np.rint(np.exp(np.log(median) + sigma * z))
    return np.clip(ln, lo, hi).astype(np.int64)


# --------------------------------------------------------------------------
# workload container
# --------------------------------------------------------------------------
@dataclass
class Workload:
    """One batch: a slot pool description, a per-token slot table and calls.

    ``calls`` lists the projection applications of one step as target ids;
    activations and weights are generated lazily and deterministically from
    ``(seed, kind, index...)`` so that large configurations never need to be
    held in host memory at once.
    """
    name: str
    config: int
    seed: int
    kind: str                                  # "bgmv" (decode) or "sgmv" (prefill / mixed)
    targets: List[Tuple[int, int]]             # (d_in, d_out) per adapted projection
    num_slots: int
    r_max: int
    ranks: np.ndarray                          # int32 [num_slots]
    scales: np.ndarray                         # float32 [num_slots]
    loaded: np.ndarray                         # int32 [num_slots] (1 = slot holds an adapter)
    slot_idx: np.ndarray                       # int32 [T], -1 = backbone-only token
    calls: List[int]                           # target id of every apply in the step
    tile_m: int = 16
    long_min: int = 128
    weight_mode: str = "lora"                  # "lora", "unitB", "int"
    act_mode: str = "normal"                   # "normal", "zero_base", "int"
    swap_victims: List[int] = field(default_factory=list)
    info: Dict[str, object] = field(default_factory=dict)

    # -- sizes ------------------------------------------------------------
    @property
    def T(self) -> int:
        return int(self.slot_idx.shape[0])

    def active_mask(self) -> np.ndarray:
        s = self.slot_idx
        ok = (s >= 0) & (s < self.num_slots)
        ok[ok] &= self.loaded[s[ok]] != 0
        return ok

    def distinct_slots(self) -> np.ndarray:
        return np.unique(self.slot_idx[self.active_mask()])

    # -- lazily generated tensors ----------------------------------------
    def _rng(self, *key: int) -> np.random.Generator:
        return np.random.default_rng([self.seed, *[int(k) for k in key]])

    def adapter_weights(self, slot: int, target: int) -> Tuple[np.ndarray, np.ndarray]:
        """(A, B) of the adapter resident in ``slot`` for ``target``.

        A: bf16 bits [d_in, r]; B: bf16 bits [r, d_out]; r = ranks[slot].
        """
        d_in, d_out = self.targets[target]
        r = int(self.ranks[slot])
        rng = self._rng(1, slot, target)
        if self.weight_mode == "int":
            # sparse small integers: every product and partial sum stays exactly representable
            A = (rng.integers(-1, 2, size=(d_in, r)) * (rng.random((d_in, r)) < 0.25)).astype(np.float32)
            B = (rng.integers(-1, 2, size=(r, d_out)) * (rng.random((r, d_out)) < 0.25)).astype(np.float32)
        else:
            lim = 1.0 / np.sqrt(d_in)
            A = rng.uniform(-lim, lim, size=(d_in, r)).astype(np.float32)
            sd = 1.0 if self.weight_mode == "unitB" else 0.02
            B = (rng.standard_normal((r, d_out)) * sd).astype(np.float32)
        return bf16_round(A), bf16_round(B)

    def activations(self, call: int, rows: Optional[np.ndarray] = None) -> Tuple[np.ndarray, np.ndarray]:
        """(x, y_base) for the ``call``-th apply of the step, bf16 bits.

        ``rows`` restricts the result to those token rows (same values as the
        full tensors would hold there).
        """
        d_in, d_out = self.targets[self.calls[call]]
        T = self.T
        rng = self._rng(2, call)
        if self.act_mode == "int":
            x = (rng.integers(-1, 2, size=(T, d_in)) * (rng.random((T, d_in)) < 0.125)).astype(np.float32)
            yb = rng.integers(-8, 9, size=(T, d_out)).astype(np.float32)
        else:
            x = rng.standard_normal((T, d_in), dtype=np.float32)
            if self.act_mode == "zero_base":
                yb = np.zeros((T, d_out), dtype=np.float32)
            else:
                yb = rng.standard_normal((T, d_out), dtype=np.float32)
        if rows is not None:
            x, yb = x[rows], yb[rows]
        return bf16_round(x), bf16_round(yb)


# --------------------------------------------------------------------------
# the five configurations
# --------------------------------------------------------------------------
LLAMA3_8B_TARGETS = [  # q, k, v, o, gate, up, down
    (4096, 4096), (4096, 1024), (4096, 1024), (4096, 4096),
    (4096, 14336), (4096, 14336), (14336, 4096),
]


def _seed(config: int, rep: int) -> int:
    return SEED_BASE + 1000 * config + rep


def make_config(config: int, rep: int = 0, layers: int = 32) -> Workload:
    """Build one of the five configurations (see module docstring)."""
    seed = _seed(config, rep)
    rng = np.random.default_rng([seed, 0])
    if config == 0:
        N, T = 8, 16
        return Workload("decode_tiny", 0, seed, "bgmv", [(1024, 1024)], N, 8,
                        np.full(N, 8, np.int32), np.full(N, 2.0, np.float32),
                        np.ones(N, np.int32), rng.integers(0, N, T).astype(np.int32), [0],
                        tile_m=8)
    if config == 1:
        N, T = 128, 256
        return Workload("decode_q_proj", 1, seed, "bgmv", [(4096, 4096)], N, 16,
                        np.full(N, 16, np.int32), np.full(N, 2.0, np.float32),
                        np.ones(N, np.int32), bounded_zipf(rng, N, 1.1, T), [0], tile_m=8)
    if config == 2:
        N, R = 64, 32
        lens = lognormal_lengths(rng, R, 512.0, 1.0, 32, 2048)
        req_slot = rng.integers(0, N, R).astype(np.int32)
        ranks = rng.choice(np.array([8, 16, 32], np.int32), size=N).astype(np.int32)
        slot_idx = np.repeat(req_slot, lens).astype(np.int32)
        return Workload("prefill_mlp", 2, seed, "sgmv", [(4096, 14336), (14336, 4096)], N, 32,
                        ranks, np.full(N, 2.0, np.float32), np.ones(N, np.int32), slot_idx,
                        [0, 1], tile_m=128, long_min=128,
                        info={"request_lengths": lens, "request_slots": req_slot})
    if config == 3:
        N = 384
        ranks = rng.choice(np.array([8, 16, 32, 64], np.int32), size=N).astype(np.int32)
        dec = bounded_zipf(rng, N, 0.9, 512)
        chunk_slot = bounded_zipf(rng, N, 0.9, 4)
        slot_idx = np.concatenate([dec, np.repeat(chunk_slot, 512)]).astype(np.int32)
        return Workload("mixed_chunked_qkv", 3, seed, "sgmv", [(4096, 6144)], N, 64,
                        ranks, np.full(N, 2.0, np.float32), np.ones(N, np.int32), slot_idx,
                        [0], tile_m=128, long_min=128, info={"chunk_slots": chunk_slot})
    if config == 4:
        N, T, n_miss = 256, 256, 16
        targets = LLAMA3_8B_TARGETS * layers
        # victims: the 16 least popular slots receive the swapped-in adapters; this
        # step's tokens draw from the Zipf over the other slots.
        victims = list(range(N - n_miss, N))
        slot_idx = bounded_zipf(rng, N - n_miss, 1.1, T)
        return Workload("llama3_8b_step", 4, seed, "bgmv", targets, N, 16,
                        np.full(N, 16, np.int32), np.full(N, 2.0, np.float32),
                        np.ones(N, np.int32), slot_idx, list(range(len(targets))),
                        tile_m=8, swap_victims=victims, info={"layers": layers})
    raise ValueError(f"unknown config {config}")


# --------------------------------------------------------------------------
# custom / adversarial batches for tests
# --------------------------------------------------------------------------
def make_custom(T: int, d_in: int, d_out: int, num_slots: int,
                ranks: Sequence[int] | int, *, seed: int = 7, r_max: Optional[int] = None,
                scale: float | Sequence[float] = 0.3, kind: str = "bgmv",
                index: str = "uniform", frac_none: float = 0.0, frac_invalid: float = 0.0,
                unloaded: Sequence[int] = (), weight_mode: str = "lora",
                act_mode: str = "normal", tile_m: int = 16, long_min: int = 128,
                slot_idx: Optional[np.ndarray] = None) -> Workload:
    """A single-target batch with controllable structure.

    index: "uniform" | "zipf" | "same" | "distinct" | "sorted" (uniform draws, sorted).
    frac_none: share of tokens set to -1; frac_invalid: share set to an
    out-of-range id (num_slots + small, or < -1).
    """
    rng = np.random.default_rng([seed, 99])
    if np.isscalar(ranks):
        rk = np.full(num_slots, int(ranks), np.int32)
    else:
        rk = np.resize(np.asarray(list(ranks), np.int32), num_slots).astype(np.int32)
    if np.isscalar(scale):
        sc = np.full(num_slots, float(scale), np.float32)
    else:
        sc = np.resize(np.asarray(list(scale), np.float32), num_slots).astype(np.float32)
    loaded = np.ones(num_slots, np.int32)
    for u in unloaded:
        loaded[u] = 0
    if slot_idx is None:
        if index == "uniform":
            s = rng.integers(0, num_slots, T)
        elif index == "sorted":
            s = np.sort(rng.integers(0, num_slots, T))
        elif index == "zipf":
            s = bounded_zipf(rng, num_slots, 1.1, T)
        elif index == "same":
            s = np.full(T, num_slots // 2)
        elif index == "distinct":
            s = rng.permutation(max(num_slots, T))[:T] % num_slots
        else:
            raise ValueError(index)
        s = s.astype(np.int32)
        if frac_none > 0:
            s[rng.random(T) < frac_none] = -1
        if frac_invalid > 0:
            bad = rng.random(T) < frac_invalid
            s[bad] = np.where(rng.random(int(bad.sum())) < 0.5, num_slots + 3, -7).astype(np.int32)
    else:
        s = np.asarray(slot_idx, np.int32)
        T = int(s.shape[0])
    return Workload("custom", -1, seed, kind, [(d_in, d_out)], num_slots,
                    int(r_max if r_max is not None else int(rk.max())), rk, sc, loaded, s, [0],
                    tile_m=tile_m, long_min=long_min, weight_mode=weight_mode, act_mode=act_mode)
