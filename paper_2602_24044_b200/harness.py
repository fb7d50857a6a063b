"""Device-side harness around the C entry points: allocates the buffers a caller owns
(PyTorch tensors), fills a slot pool from a workload and runs applies.  Used by the GPU
tests, the smoke check and the benchmark.  No arithmetic of the method lives here.
"""
from __future__ import annotations

from typing import Dict, List, Optional, Sequence

import numpy as np
import torch

from . import binding as lb


def bf16_tensor(bits: np.ndarray, device=None, pin: bool = False) -> torch.Tensor:
    """numpy uint16 bf16 bit patterns -> torch.bfloat16 tensor (same bits)."""
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16)
    if pin:
        t = t.pin_memory()
    if device is not None:
        t = t.to(device, non_blocking=False)
    return t


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    """torch.bfloat16 tensor -> numpy uint16 bit patterns (waits for all queued GPU work)."""
    if t.is_cuda:
        torch.cuda.synchronize(t.device)
    return t.detach().contiguous().cpu().view(torch.int16).numpy().view(np.uint16)


class Session:
    """A slot pool on one GPU filled from a workload, plus per-batch scratch buffers."""

    def __init__(self, wl, device: str = "cuda:0", targets: Optional[Sequence[int]] = None,
                 slots: Optional[Sequence[int]] = None, a_layout: int = lb.A_DIN_MAJOR,
                 T_cap: Optional[int] = None, tuning: Optional[Dict[int, int]] = None):
        """targets: the workload's target ids to materialise in the pool (default: all);
        slots: which occupied slots to load (default: every slot the workload marks loaded)."""
        self.wl = wl
        self.device = torch.device(device)
        self.dev_index = self.device.index or 0
        self.target_ids = list(range(len(wl.targets))) if targets is None else list(targets)
        self.pool_targets = [wl.targets[t] for t in self.target_ids]
        self.target_pos = {t: i for i, t in enumerate(self.target_ids)}
        torch.cuda.set_device(self.device)
        self.compute = torch.cuda.Stream(self.device)
        self.load = torch.cuda.Stream(self.device)
        nbytes = lb.pool_bytes(wl.num_slots, wl.r_max, self.pool_targets, self.dev_index)
        self.pool_buf = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
        off = (-self.pool_buf.data_ptr()) % 256
        self.pool_mem = self.pool_buf[off:off + nbytes]
        self.pool = lb.pool_create(wl.num_slots, wl.r_max, self.pool_targets, self.pool_mem,
                                   self.dev_index)
        for key, value in (tuning or {}).items():
            lb.pool_set_tuning(self.pool, key, value)
        self.T_cap = int(T_cap if T_cap is not None else max(wl.T, 1))
        self.ws = torch.empty(lb.workspace_bytes(self.pool, self.T_cap), dtype=torch.uint8,
                              device=self.device)
        self.meta = None
        self.meta_shape = None
        self.slot_idx_dev = torch.from_numpy(np.ascontiguousarray(wl.slot_idx)).to(self.device)
        self.status_host = torch.zeros(4, dtype=torch.int32).pin_memory()
        self._pinned: List[torch.Tensor] = []
        want = [i for i in range(wl.num_slots) if wl.loaded[i]] if slots is None else list(slots)
        for s in want:
            self.load_slot(s, a_layout=a_layout)
        torch.cuda.synchronize(self.device)
        self._pinned.clear()

    # -- pool ----------------------------------------------------------------------------
    def host_adapter(self, slot: int, a_layout: int):
        """Pinned host matrices of one adapter for the pool's targets."""
        A, B = [], []
        for t in self.target_ids:
            a, b = self.wl.adapter_weights(slot, t)
            if a_layout == lb.A_RANK_MAJOR:
                a = np.ascontiguousarray(a.T)
            A.append(bf16_tensor(a, pin=True))
            B.append(bf16_tensor(b, pin=True))
        return A, B

    def host_adapter_packed(self, slot: int):
        """One pinned buffer with every target's A [rank, d_in] and B [rank, d_out] in order."""
        parts = []
        for t in self.target_ids:
            a, b = self.wl.adapter_weights(slot, t)
            parts += [np.ascontiguousarray(a.T).ravel(), np.ascontiguousarray(b).ravel()]
        buf = bf16_tensor(np.concatenate(parts), pin=True)
        return [buf] * len(self.target_ids), [buf] * len(self.target_ids)

    def load_slot(self, slot: int, a_layout: int = lb.A_DIN_MAJOR, src_slot: Optional[int] = None,
                  rank: Optional[int] = None, scale: Optional[float] = None, blobs=None):
        """Queue a swap-in of the workload's adapter `src_slot` (default: `slot`) into `slot`."""
        src = slot if src_slot is None else src_slot
        if blobs is not None:
            A, B = blobs
        elif a_layout == lb.PACKED:
            A, B = self.host_adapter_packed(src)
        else:
            A, B = self.host_adapter(src, a_layout)
        self._pinned += A + B
        lb.pool_load_slot(self.pool, slot, int(self.wl.ranks[src]) if rank is None else rank,
                          float(self.wl.scales[src]) if scale is None else scale, A, B, a_layout,
                          self.load, self.compute)

    def read_slot(self, slot: int, target: int):
        d_in, d_out = self.wl.targets[target]
        A = torch.empty((self.wl.r_max, d_in), dtype=torch.bfloat16).pin_memory()
        B = torch.empty((self.wl.r_max, d_out), dtype=torch.bfloat16).pin_memory()
        lb.pool_read_slot(self.pool, slot, self.target_pos[target], A, B, self.compute)
        self.compute.synchronize()
        return bf16_bits(A), bf16_bits(B)

    def status(self) -> np.ndarray:
        lb.pool_poll_status(self.pool, self.status_host, self.compute)
        self.compute.synchronize()
        return self.status_host.numpy().copy()

    # -- metadata ------------------------------------------------------------------------
    def build_segments(self, tile_m: Optional[int] = None, long_min: Optional[int] = None,
                       slot_idx_dev: Optional[torch.Tensor] = None):
        wl = self.wl
        tile_m = wl.tile_m if tile_m is None else tile_m
        long_min = wl.long_min if long_min is None else long_min
        sidx = self.slot_idx_dev if slot_idx_dev is None else slot_idx_dev
        T = int(sidx.shape[0])
        nbytes = lb.segments_bytes(T, wl.num_slots, tile_m)
        if self.meta is None or self.meta.numel() * 4 < nbytes:
            self.meta = torch.empty((nbytes + 3) // 4, dtype=torch.int32, device=self.device)
        lb.build_segments(self.pool, sidx, T, tile_m, long_min, self.meta, stream=self.compute)
        self.meta_shape = (T, tile_m)
        return self.meta

    def segments_host(self) -> Dict[str, np.ndarray]:
        self.compute.synchronize()
        T, tile_m = self.meta_shape
        return lb.unpack_segments(self.meta.cpu().numpy(), T, self.wl.num_slots, tile_m)

    # -- the forward ---------------------------------------------------------------------
    def apply(self, call: int = 0, x: Optional[torch.Tensor] = None,
              y_base: Optional[torch.Tensor] = None, *, kind: Optional[str] = None,
              grouped: bool = True, in_place: bool = False,
              slot_idx_dev: Optional[torch.Tensor] = None, rebuild: bool = True,
              ws_bytes: Optional[int] = None) -> torch.Tensor:
        """One apply on the compute stream; returns y (device tensor).  x / y_base default to
        the workload's activations for `call`.  ws_bytes: how much of the workspace the call is
        told about (default: all of it)."""
        wl = self.wl
        target = wl.calls[call]
        d_in, d_out = wl.targets[target]
        if x is None:
            x_h, yb_h = wl.activations(call)
            x, y_base = bf16_tensor(x_h, self.device), bf16_tensor(yb_h, self.device)
        T = int(x.shape[0])
        kind = wl.kind if kind is None else kind
        sidx = self.slot_idx_dev if slot_idx_dev is None else slot_idx_dev
        y = y_base if in_place else torch.empty_like(y_base)
        with torch.cuda.stream(self.compute):
            if not in_place:
                # a row the kernels never write must not pass for a result left over in recycled
                # memory: the output starts as a huge finite value in every element
                y.view(torch.int16).fill_(0x7F7F)
            meta = None
            if grouped or kind == "sgmv":
                if rebuild or self.meta_shape is None:
                    self.build_segments(slot_idx_dev=sidx)
                meta = self.meta
            tp = self.target_pos[target]
            if kind == "bgmv":
                lb.bgmv_apply(self.pool, tp, x, x.stride(0), y_base, y_base.stride(0), y,
                              y.stride(0), sidx, T, meta, self.ws, stream=self.compute)
            else:
                lb.sgmv_apply(self.pool, tp, x, x.stride(0), y_base, y_base.stride(0), y,
                              y.stride(0), meta, T, self.ws, ws_bytes, stream=self.compute)
        return y

    def close(self):
        if self.pool:
            torch.cuda.synchronize(self.device)
            lb.pool_destroy(self.pool)
            self.pool = 0

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()
