"""The failure-detection path: a bounded device-side wait that runs out is reported as HTS_ERR_TIMEOUT,
the kernel returns by itself and the context keeps working (no fault, no hang: the wait has a limit)."""
import numpy as np
import pytest
import torch

import hts_workloads as wl
import paper_2012_09849_b200 as hts
from oracle import hts_oracle as orc
from gpu_util import Policy, rel_err

pytestmark = pytest.mark.gpu


def test_expired_wait_is_reported_once_and_the_context_survives():
    cfg = wl.CONFIGS[2]
    pol = Policy(cfg, max_batch=32)
    try:
        n = 20
        obs = wl.make_obs(cfg, n, batch_index=3)
        ids = np.arange(n, dtype=np.int32)
        before = pol.step(obs, ids, 1, 77)
        assert hts.hts_last_async_error(pol.ctx) == 0
        hts.hts_wait_selftest(pol.ctx, 100_000)          # ~50 microseconds of waiting on a barrier nobody signals
        torch.cuda.synchronize()                         # the kernel has returned by itself
        assert hts.hts_last_async_error(pol.ctx) == 5    # HTS_ERR_TIMEOUT
        assert hts.hts_last_async_error(pol.ctx) == 0    # reading clears it
        after = pol.step(obs, ids, 1, 77)                # the context still works, bit for bit
        for k in before:
            assert np.array_equal(before[k].view(np.int32), after[k].view(np.int32)), k
        ref = orc.policy_step(orc.Weights(pol.params), obs, ids, 1, 77)
        assert rel_err(after["logits"], ref["logits"]) <= 2e-2
        assert rel_err(after["values"], ref["values"]) <= 2e-2
    finally:
        pol.close()


def test_selftest_arguments_are_checked_on_the_host():
    cfg = wl.CONFIGS[2]
    pol = Policy(cfg, max_batch=4)
    try:
        for bad in (0, 999, 10**9):
            with pytest.raises(hts.HtsError) as e:
                hts.hts_wait_selftest(pol.ctx, bad)
            assert e.value.status == 1
    finally:
        pol.close()
