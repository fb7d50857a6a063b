"""GPU tests of the slot pool's swap-in path and of the host-buffer entry point."""
import numpy as np
import pytest

from gpu_util import check_tolerance, oracle_full, require_gpu
from oracle import lora_oracle as orc
from paper_2602_24044_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _gpu():
    require_gpu()


def _bits(t):
    from paper_2602_24044_b200.harness import bf16_bits
    return bf16_bits(t)


def test_swap_in_does_not_disturb_an_apply_in_flight_then_takes_effect():
    import torch
    from paper_2602_24044_b200 import binding as lb
    from paper_2602_24044_b200.harness import Session, bf16_tensor
    wl = W.make_custom(512, 2048, 2048, 16, 16, scale=0.9, index="uniform", seed=3)
    x_h, yb_h = wl.activations(0)
    with Session(wl) as s:
        x, yb = bf16_tensor(x_h, s.device), bf16_tensor(yb_h, s.device)
        before = _bits(s.apply(x=x, y_base=yb))
        # queue applies, then immediately a swap of every slot to another adapter's weights on
        # the load stream; the load must wait for the queued readers
        ys = [s.apply(x=x, y_base=yb, rebuild=False) for _ in range(4)]
        for slot in range(16):
            s.load_slot(slot, src_slot=(slot + 1) % 16, scale=1.3)
        for y in ys:
            assert np.array_equal(_bits(y), before)
        # the swapped adapters become visible after acquire
        lb.pool_acquire(s.pool, list(range(16)), s.compute)
        after = _bits(s.apply(x=x, y_base=yb))
        torch.cuda.synchronize()
        A = [W.bf16_to_f64(wl.adapter_weights((i + 1) % 16, 0)[0]) for i in range(16)]
        B = [W.bf16_to_f64(wl.adapter_weights((i + 1) % 16, 0)[1]) for i in range(16)]
        y_ref, _ = orc.apply(W.bf16_to_f64(x_h), W.bf16_to_f64(yb_h), wl.slot_idx, A, B, wl.ranks,
                             np.full(16, np.float32(1.3), np.float64), wl.loaded, threads=8)
        check_tolerance(after, y_ref, what="after swap")
        assert not np.array_equal(after, before)
        assert lb.pool_slot_info(s.pool, 3) == (16, pytest.approx(1.3))


def test_evicted_slot_is_treated_as_no_adapter():
    from paper_2602_24044_b200 import binding as lb
    from paper_2602_24044_b200.harness import Session
    wl = W.make_custom(64, 256, 256, 4, 8, seed=5)
    _, yb_h = wl.activations(0)
    with Session(wl) as s:
        lb.pool_evict_slot(s.pool, 2, s.load, s.compute)
        lb.pool_acquire(s.pool, [2], s.compute)
        loaded = wl.loaded.copy()
        loaded[2] = 0
        for grouped in (True, False):
            lb.pool_reset_status(s.pool, s.compute)
            y = _bits(s.apply(grouped=grouped))
            hit = wl.slot_idx == 2
            assert np.array_equal(y[hit], yb_h[hit])
            assert s.status()[0] == int(hit.sum())
        assert lb.pool_slot_info(s.pool, 2)[0] == 0


def test_load_slot_argument_errors_leave_the_slot_untouched():
    import torch
    from paper_2602_24044_b200 import binding as lb
    from paper_2602_24044_b200.harness import Session
    wl = W.make_custom(8, 64, 64, 2, 8, seed=6)
    with Session(wl) as s:
        A0, B0 = s.read_slot(1, 0)
        A, B = s.host_adapter(0, lb.A_DIN_MAJOR)
        pageable = np.zeros((64, 8), np.uint16)
        for kwargs, status in [
            (dict(slot=5, rank=8, A=A, B=B), 3),
            (dict(slot=-1, rank=8, A=A, B=B), 3),
            (dict(slot=1, rank=9, A=A, B=B), 4),
            (dict(slot=1, rank=0, A=A, B=B), 4),
            (dict(slot=1, rank=8, A=[pageable], B=B), 8),
            (dict(slot=1, rank=8, A=A, B=B, a_layout=7), 1),
        ]:
            with pytest.raises(lb.LoraError) as e:
                lb.pool_load_slot(s.pool, scale=1.0, load_stream=s.load, compute_stream=s.compute,
                                  **kwargs)
            assert e.value.status == status, kwargs
        torch.cuda.synchronize()
        A1, B1 = s.read_slot(1, 0)
        assert np.array_equal(A0, A1) and np.array_equal(B0, B1)
        assert lb.pool_slot_info(s.pool, 1)[0] == 8


def test_apply_argument_errors():
    import torch
    from paper_2602_24044_b200 import binding as lb
    from paper_2602_24044_b200.harness import Session
    wl = W.make_custom(8, 64, 64, 2, 8, seed=7)
    with Session(wl) as s:
        x = torch.zeros((8, 64), dtype=torch.bfloat16, device=s.device)
        yb = torch.zeros((8, 64), dtype=torch.bfloat16, device=s.device)
        y = torch.zeros((8, 64), dtype=torch.bfloat16, device=s.device)
        big = torch.zeros((9, 64), dtype=torch.bfloat16, device=s.device)

        def call(**kw):
            a = dict(target=0, x=x, ldx=64, y_base=yb, ldyb=64, y=y, ldy=64,
                     slot_idx_dev=s.slot_idx_dev, T=8, meta_dev=None, workspace=s.ws)
            a.update(kw)
            lb.bgmv_apply(s.pool, stream=s.compute, **a)

        call()
        for kw, status in [(dict(target=1), 3), (dict(T=-1), 2), (dict(ldx=60), 2),
                           (dict(ldyb=68), 2), (dict(x=None), 1),
                           (dict(y_base=big, y=big.reshape(-1)[32:]), 1),     # partial overlap
                           (dict(workspace=s.ws[:64]), 7),
                           (dict(slot_idx_dev=None), 1),
                           (dict(meta_dev=s.ws), 1)]:                         # not a built table
            with pytest.raises(lb.LoraError) as e:
                call(**kw)
            assert e.value.status == status, kw
        torch.cuda.synchronize()


@pytest.mark.parametrize("kind", [0, 1])
def test_host_buffer_entry_point_matches_oracle(kind):
    import torch
    from paper_2602_24044_b200 import binding as lb
    from paper_2602_24044_b200.harness import Session, bf16_tensor
    wl = W.make_custom(300, 512, 768, 12, [8, 16, 32], index="zipf", frac_none=0.1, seed=8,
                       tile_m=16 if kind == 0 else 128)
    y_ref, _ = oracle_full(wl)
    x_h, yb_h = wl.activations(0)
    with Session(wl) as s:
        xh, ybh = bf16_tensor(x_h, pin=True), bf16_tensor(yb_h, pin=True)
        yh = torch.empty_like(ybh).pin_memory()
        sh = torch.from_numpy(wl.slot_idx.copy()).pin_memory()
        xd = torch.empty((300, 512), dtype=torch.bfloat16, device=s.device)
        ybd = torch.empty((300, 768), dtype=torch.bfloat16, device=s.device)
        yd = torch.empty_like(ybd)
        sd = torch.empty(300, dtype=torch.int32, device=s.device)
        meta = torch.empty(lb.segments_bytes(300, 12, wl.tile_m) // 4, dtype=torch.int32,
                           device=s.device)
        lb.apply_host(s.pool, 0, kind, xh, ybh, yh, sh, 300, wl.tile_m, 128, xd, ybd, yd, sd, meta,
                      s.ws, s.compute)
        s.compute.synchronize()
        check_tolerance(_bits(yh), y_ref, what="host entry point")


@pytest.mark.parametrize("rank,r_max", [(16, 16), (8, 16)])
def test_packed_adapter_lands_in_the_slot_layout(rank, r_max):
    """One pinned buffer per adapter (LORA_PACKED): the slot holds the same bytes as after a
    matrix-by-matrix load, padding rows are zero, and the forward matches the oracle."""
    from paper_2602_24044_b200 import binding as lb
    from paper_2602_24044_b200.harness import Session
    wl = W.make_custom(96, 256, 512, 4, rank, r_max=r_max, scale=0.7, index="uniform", seed=21)
    wl.targets = wl.targets + [(512, 128)]
    y_ref, _ = oracle_full(wl)
    with Session(wl, slots=[]) as s:
        for slot in range(4):
            s.load_slot(slot, a_layout=lb.PACKED)
        lb.pool_acquire(s.pool, list(range(4)), s.compute)
        for slot in range(4):
            for t in range(2):
                A, B = s.read_slot(slot, t)
                a, b = wl.adapter_weights(slot, t)
                assert np.array_equal(A[:rank], a.T) and np.array_equal(B[:rank], b)
                assert not A[rank:].any() and not B[rank:].any()
        check_tolerance(_bits(s.apply()), y_ref, what="packed load")
