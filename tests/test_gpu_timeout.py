"""The time-out path on the device: a bounded wait that runs out is recorded in the pool's status
word 1, nothing is stored, the context stays usable, and the synchronous status check turns the
word into LORA_ERR_TIMEOUT.  The wait is made to run out by a one-block kernel whose barrier
nobody completes (a small poll limit); no kernel is made to hang or fault."""
import numpy as np
import pytest

from gpu_util import check_tolerance, oracle_full, require_gpu
from paper_2602_24044_b200 import workloads as W

pytestmark = pytest.mark.gpu


def test_expired_wait_is_reported_and_the_pool_keeps_working():
    require_gpu()
    import torch
    from paper_2602_24044_b200 import binding as lb
    from paper_2602_24044_b200.harness import Session, bf16_bits
    wl = W.make_custom(40, 512, 256, 4, 16, scale=1.1, weight_mode="unitB", seed=61)
    y_ref, _ = oracle_full(wl)
    with Session(wl) as s:
        assert lb.pool_check_status(s.pool, s.compute) == [0, 0, 0, 0]
        witness = torch.full((1,), 7, dtype=torch.int32, device=s.device)
        lb.pool_selftest_wait_expiry(s.pool, 1 << 10, witness, s.compute)
        assert s.status()[1] == 1                      # recorded
        assert int(witness.item()) == 7                # and nothing stored
        with pytest.raises(lb.LoraError) as e:
            lb.pool_check_status(s.pool, s.compute)
        assert e.value.status == 10
        lb.pool_selftest_wait_expiry(s.pool, 1, None, s.compute)
        assert s.status()[1] == 2                      # expiries accumulate until the reset
        lb.pool_reset_status(s.pool, s.compute)
        assert lb.pool_check_status(s.pool, s.compute) == [0, 0, 0, 0]
        # the context and the pool are intact: a normal apply afterwards matches the oracle
        check_tolerance(bf16_bits(s.apply()), y_ref, what="apply after an expired wait")
        assert lb.pool_check_status(s.pool, s.compute)[1] == 0
        for bad in (0, (1 << 20) + 1):
            with pytest.raises(lb.LoraError) as e:
                lb.pool_selftest_wait_expiry(s.pool, bad, None, s.compute)
            assert e.value.status == 1
