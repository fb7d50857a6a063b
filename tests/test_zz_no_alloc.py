"""The workspace-free decode entry point (collected last on purpose: a run that stops at the
first failure has then already been through every other test).

lora_bgmv_apply_static exists for hosts that cannot allocate device memory where they call the
library (all HBM already handed to a KV cache and the adapter pool, or running under another
framework's allocator): its scratch is a fixed array inside the library.  Here it is called
through the C ABI twice in a row and compared with lora_bgmv_apply on the same inputs, and with
the CPU oracle at the bound the other path tests use."""
import numpy as np
import pytest

from gpu_util import check_tolerance, require_gpu
from oracle import lora_oracle as orc
from paper_2602_24044_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _within_tolerance(a_bits, b_bits):
    a, b = W.bf16_to_f64(a_bits), W.bf16_to_f64(b_bits)
    return bool(np.all(np.abs(a - b) <= 1e-2 * np.abs(b) + 1e-2))


@pytest.mark.parametrize("grouped", [True, False])
def test_static_scratch_entry_point_matches_workspace_entry_point(grouped):
    require_gpu()
    import torch
    from paper_2602_24044_b200 import binding as lb
    from paper_2602_24044_b200.harness import Session, bf16_bits, bf16_tensor
    wl = W.make_custom(200, 1024, 768, 24, [4, 8, 16], scale=[0.3, 1.7], index="zipf",
                       frac_none=0.1, frac_invalid=0.05, weight_mode="unitB", seed=21)
    with Session(wl) as s:
        T = wl.T
        for call in range(2):                      # two calls in a row share the library's array
            x_h, yb_h = W.make_custom(200, 1024, 768, 24, [4, 8, 16], seed=30 + call,
                                      weight_mode="unitB").activations(0)
            x, yb = bf16_tensor(x_h, s.device), bf16_tensor(yb_h, s.device)
            want = bf16_bits(s.apply(x=x, y_base=yb, grouped=grouped))
            y = torch.empty_like(yb)
            meta = s.meta if grouped else None
            lb.bgmv_apply_static(s.pool, 0, x, 1024, yb, 768, y, 768, s.slot_idx_dev, T, meta,
                                 s.compute)
            got = bf16_bits(y)
            assert _within_tolerance(got, want), "call %d" % call
            y_ref, _ = orc.apply_workload(wl, 0, threads=4, acts=(x_h, yb_h))
            check_tolerance(got, y_ref, what="static entry point, call %d" % call)
            idle = ~wl.active_mask()
            assert np.array_equal(got[idle], yb_h[idle])
        # in place as well
        yb2 = yb.clone()
        lb.bgmv_apply_static(s.pool, 0, x, 1024, yb2, 768, yb2, 768, s.slot_idx_dev, T, meta,
                             s.compute)
        assert _within_tolerance(bf16_bits(yb2), want)
        check_tolerance(bf16_bits(yb2), y_ref, what="static entry point, in place")
        assert s.status()[1] == 0                  # no bounded device-side wait expired


def test_static_scratch_entry_point_rejects_oversized_batches():
    require_gpu()
    import torch
    from paper_2602_24044_b200 import binding as lb
    from paper_2602_24044_b200.harness import Session
    # r_max 64: the limit is 32 * T * 64 <= 2 MiB, i.e. T <= 1024
    wl = W.make_custom(8, 64, 64, 2, 64, seed=22)
    with Session(wl) as s:
        T = 1025
        x = torch.zeros((T, 64), dtype=torch.bfloat16, device=s.device)
        yb = torch.zeros((T, 64), dtype=torch.bfloat16, device=s.device)
        sidx = torch.zeros(T, dtype=torch.int32, device=s.device)
        before = lb.launch_count()
        with pytest.raises(lb.LoraError) as e:
            lb.bgmv_apply_static(s.pool, 0, x, 64, yb, 64, yb, 64, sidx, T, None, s.compute)
        assert e.value.status == 7 and lb.launch_count() == before
        lb.bgmv_apply_static(s.pool, 0, x[:1024], 64, yb[:1024], 64, yb[:1024], 64, sidx, 1024, None,
                             s.compute)
        torch.cuda.synchronize()
    # r_max 16: T <= 4096
    wl16 = W.make_custom(8, 64, 64, 2, 16, seed=23)
    with Session(wl16) as s, Session(wl16) as s2:
        T = 4097
        x = torch.zeros((T, 64), dtype=torch.bfloat16, device=s.device)
        yb = torch.zeros((T, 64), dtype=torch.bfloat16, device=s.device)
        sidx = torch.zeros(T, dtype=torch.int32, device=s.device)
        with pytest.raises(lb.LoraError) as e:
            lb.bgmv_apply_static(s.pool, 0, x, 64, yb, 64, yb, 64, sidx, T, None, s.compute)
        assert e.value.status == 7
        # two pools on one device use the same array, one after the other
        for sess in (s, s2):
            lb.bgmv_apply_static(sess.pool, 0, x[:4096], 64, yb[:4096], 64, yb[:4096], 64, sidx, 4096,
                                 None, sess.compute)
            torch.cuda.synchronize()
            assert sess.status()[1] == 0
