"""Several projections of one decode batch in one launch (lora_bgmv_apply_multi): every projection
against the fp64 oracle, bit identity with the single-projection calls, shared inputs, argument
errors; and isolation between adapters when one of them holds non-finite weights."""
import numpy as np
import pytest

from gpu_util import check_tolerance, require_gpu
from oracle import lora_oracle as orc
from paper_2602_24044_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _gpu():
    require_gpu()


def _layer_inputs(wl, s, share=True):
    """Device tensors of one layer's seven projections; q/k/v share x, gate/up share x."""
    from paper_2602_24044_b200.harness import bf16_tensor
    host, dev = [], []
    src = {1: 0, 2: 0, 5: 4} if share else {}
    for c in range(len(wl.calls)):
        x_h, yb_h = wl.activations(c)
        if c in src:
            x_h = host[src[c]][0]
        host.append((x_h, yb_h))
    for c, (x_h, yb_h) in enumerate(host):
        x = dev[src[c]][0] if c in src else bf16_tensor(x_h, s.device)
        dev.append((x, bf16_tensor(yb_h, s.device)))
    return host, dev


@pytest.mark.parametrize("tuning", [{}, {3: 3}, {5: 3, 9: 50}], ids=["default", "3-clusters", "3-stages-half"])
def test_layer_in_one_launch_matches_oracle_and_single_calls(tuning):
    import torch
    from paper_2602_24044_b200 import binding as lb
    from paper_2602_24044_b200.harness import Session, bf16_bits
    wl = W.make_config(4, layers=1)
    T = wl.T
    with Session(wl, a_layout=lb.A_RANK_MAJOR, tuning=tuning) as s:
        host, dev = _layer_inputs(wl, s)
        s.build_segments()
        single = []
        for c, (x, yb) in enumerate(dev):
            y = torch.empty_like(yb)
            lb.bgmv_apply(s.pool, c, x, x.shape[1], yb, yb.shape[1], y, y.shape[1], s.slot_idx_dev, T,
                          s.meta, s.ws, stream=s.compute)
            single.append(y)
        # widest projections first: gate, up, down, q, o, k, v
        order = [4, 5, 6, 0, 3, 1, 2]
        outs = {c: torch.zeros_like(dev[c][1]) for c in order}
        items = [(c, dev[c][0], dev[c][0].shape[1], dev[c][1], dev[c][1].shape[1], outs[c],
                  outs[c].shape[1]) for c in order]
        for _ in range(2):          # the second launch reads the table ahead of its predecessor's end
            lb.bgmv_apply_multi(s.pool, items, s.slot_idx_dev, T, s.meta, s.ws, stream=s.compute)
        torch.cuda.synchronize()
        for c in order:
            got = bf16_bits(outs[c])
            assert np.array_equal(got, bf16_bits(single[c])), "projection %d differs from the single call" % c
            y_ref, _ = orc.apply_workload(wl, c, threads=8, acts=host[c])
            check_tolerance(got, y_ref, what="multi, projection %d" % c)
        assert s.status()[1] == 0


def test_mixed_ranks_idle_rows_and_in_place_items():
    import torch
    from paper_2602_24044_b200 import binding as lb
    from paper_2602_24044_b200.harness import Session, bf16_bits, bf16_tensor
    wl = W.make_custom(150, 1160, 2056, 20, [1, 5, 8, 16, 24, 32, 48, 64], scale=[0.3, 1.7],
                       index="zipf", frac_none=0.1, frac_invalid=0.05, weight_mode="unitB", seed=71)
    wl.targets = [(1160, 2056), (1160, 520), (264, 2056)]
    wl.calls = [0, 1, 2]
    with Session(wl) as s:
        s.build_segments()
        items, host, outs = [], [], []
        for c in range(3):
            x_h, yb_h = wl.activations(c)
            x, yb = bf16_tensor(x_h, s.device), bf16_tensor(yb_h, s.device)
            y = yb if c == 1 else torch.empty_like(yb)          # item 1 in place
            items.append((c, x, x.shape[1], yb, yb.shape[1], y, y.shape[1]))
            host.append((x_h, yb_h))
            outs.append(y)
        lb.bgmv_apply_multi(s.pool, items, s.slot_idx_dev, wl.T, s.meta, s.ws, stream=s.compute)
        torch.cuda.synchronize()
        idle = ~wl.active_mask()
        for c in range(3):
            y_ref, n_inv = orc.apply_workload(wl, c, threads=8, acts=host[c])
            got = bf16_bits(outs[c])
            check_tolerance(got, y_ref, what="multi mixed ranks, item %d" % c)
            assert np.array_equal(got[idle], host[c][1][idle])
        assert s.status()[1] == 0


def test_multi_argument_errors():
    import torch
    from paper_2602_24044_b200 import binding as lb
    from paper_2602_24044_b200.harness import Session
    wl = W.make_custom(32, 256, 256, 4, 8, seed=72)
    wl.targets = [(256, 256)] * 2
    wl.calls = [0, 1]
    with Session(wl) as s:
        s.build_segments()
        x = torch.zeros((32, 256), dtype=torch.bfloat16, device=s.device)
        a, b = torch.zeros_like(x), torch.zeros_like(x)
        ok = [(0, x, 256, a, 256, a, 256), (1, x, 256, b, 256, b, 256)]
        before = lb.launch_count()
        for items, status in [([], 1), (ok * 5, 1),
                              ([ok[0], (1, x, 256, b, 256, a, 256)], 1),      # two items write one y
                              ([ok[0], (1, a, 256, b, 256, b, 256)], 1),      # item 1 reads what item 0 writes
                              ([(2, x, 256, a, 256, a, 256)], 3)]:
            with pytest.raises(lb.LoraError) as e:
                lb.bgmv_apply_multi(s.pool, items, s.slot_idx_dev, 32, s.meta, s.ws, stream=s.compute)
            assert e.value.status == status
        with pytest.raises(lb.LoraError) as e:      # the grouped table is required
            lb.bgmv_apply_multi(s.pool, ok, s.slot_idx_dev, 32, None, s.ws, stream=s.compute)
        assert e.value.status == 1
        assert lb.launch_count() == before
        lb.bgmv_apply_multi(s.pool, ok, s.slot_idx_dev, 32, s.meta, s.ws, stream=s.compute)
        torch.cuda.synchronize()


@pytest.mark.parametrize("clusters", [0, 1])
def test_non_finite_weights_of_one_adapter_do_not_reach_other_tokens(clusters):
    """An adapter whose B holds Inf / NaN spoils its own tokens only.  One cluster walks every
    unit (tuning key 3 = 1), so tiles of the bad rank-16 adapter and of rank-8 adapters pass
    through the same shared-memory stages one after the other."""
    from paper_2602_24044_b200.harness import Session, bf16_bits
    base = W.make_custom(96, 512, 512, 6, [16, 8, 3, 16, 8, 12], scale=0.7, index="uniform",
                         weight_mode="unitB", tile_m=8, seed=73)
    bad = 0
    plain = base.adapter_weights

    def poisoned(slot, target):
        A, B = plain(slot, target)
        if slot == bad:
            B = B.copy()
            B[8:, ::3] = 0x7F80          # +Inf
            B[9:, 1::5] = 0x7FC0         # NaN
        return A, B

    base.adapter_weights = poisoned
    y_ref, _ = orc.apply_workload(base, threads=4)
    clean = base.slot_idx != bad
    assert np.isfinite(y_ref[clean]).all() and not np.isfinite(y_ref[~clean]).all()
    for grouped in (True, False):
        with Session(base, tuning={3: clusters} if clusters else {}) as s:
            y = bf16_bits(s.apply(grouped=grouped))
            check_tolerance(y[clean], y_ref[clean], what="tokens of the clean adapters")
