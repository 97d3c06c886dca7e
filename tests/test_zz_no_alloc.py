"""The allocation-free actor step against the regular one (collected last on purpose).

Some callers cannot call cudaMalloc: their device memory belongs to another allocator, or they
sit in a loop that must not hit the device-wide synchronisation an allocation implies.
hts_policy_step_noalloc serves them from a fixed scratch array inside the library.  Here it must
reproduce, bit for bit, what hts_policy_step computes with an fp32 context on the same inputs,
twice in a row (the second call finds the first call's leftovers in the shared scratch)."""
import numpy as np
import pytest
import torch

import hts_workloads as wl
import paper_2012_09849_b200 as hts
from gpu_util import Policy

pytestmark = pytest.mark.gpu


def _noalloc(cfg, dev_w, obs, ids, t, seed):
    n = obs.shape[0]
    d_obs, d_ids = torch.from_numpy(obs).cuda(), torch.from_numpy(ids).cuda()
    act = torch.empty(n, dtype=torch.int32, device="cuda")
    logp, val, ent = (torch.empty(n, dtype=torch.float32, device="cuda") for _ in range(3))
    logits = torch.empty(n, cfg.A, dtype=torch.float32, device="cuda")
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()            # device-wide: a cudaMalloc in the library would show here
    hts.hts_policy_step_noalloc(cfg.C, cfg.H, cfg.W, cfg.A, dev_w, d_obs, d_ids, None, t, seed, n,
                                act, logp, val, ent, logits)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] >= free_before, "the call took device memory"
    return {"actions": act.cpu().numpy(), "logp": logp.cpu().numpy(), "values": val.cpu().numpy(),
            "entropy": ent.cpu().numpy(), "logits": logits.cpu().numpy()}


def test_noalloc_step_matches_regular_step_twice_in_a_row():
    cfg = wl.CONFIGS[1]                                   # fp32 weights, 4x84x84, 6 actions
    pol = Policy(cfg, max_batch=48)
    try:
        for call, (n, t) in enumerate(((16, 3), (37, 4))):   # a second, larger call reuses the scratch
            obs = wl.make_obs(cfg, n, batch_index=100 + call)
            ids = np.arange(500, 500 + n, dtype=np.int32)
            ref = pol.step(obs, ids, t, seed=99)
            got = _noalloc(cfg, pol.dev_w, obs, ids, t, 99)
            for k in ref:
                assert np.array_equal(got[k].view(np.int32), ref[k].view(np.int32)), (call, k)
    finally:
        pol.close()


def test_noalloc_step_refuses_what_does_not_fit():
    cfg = wl.CONFIGS[1]
    pol = Policy(cfg, max_batch=4)
    try:
        n = 49                                            # one more than the 4 MiB scratch holds at this shape
        obs = torch.zeros(n, cfg.C, cfg.H, cfg.W, dtype=torch.uint8, device="cuda")
        ids = torch.zeros(n, dtype=torch.int32, device="cuda")
        act = torch.zeros(n, dtype=torch.int32, device="cuda")
        f = [torch.zeros(n, device="cuda") for _ in range(3)]
        with pytest.raises(hts.HtsError) as e:
            hts.hts_policy_step_noalloc(cfg.C, cfg.H, cfg.W, cfg.A, pol.dev_w, obs, ids, None, 0, 1, n, act, *f)
        assert e.value.status == 1
        bf = hts.weights_to_device(pol.params, hts.HTS_DTYPE_BF16)
        d = hts.hts_net_desc(cfg.C, cfg.H, cfg.W, cfg.A, hts.HTS_DTYPE_BF16, 4)     # bf16 weights are not served
        w = hts.hts_weights(**{k: bf[k].data_ptr() for k in hts.WEIGHT_NAMES})
        import ctypes
        rc = hts.lib().hts_policy_step_noalloc(ctypes.byref(d), ctypes.byref(w), obs.data_ptr(), ids.data_ptr(), None,
                                               0, 1, 4, act.data_ptr(), f[0].data_ptr(), f[1].data_ptr(),
                                               f[2].data_ptr(), None, None)
        assert rc == 6
    finally:
        pol.close()
