"""The two-stream rollout schedule (actor steps of rollout k+1 overlapping the advantage scan of rollout k)
against the oracle, through the C ABI, in the schedule bench.py times."""
import numpy as np
import pytest
import torch

import hts_workloads as wl
import paper_2012_09849_b200 as hts
from paper_2012_09849_b200.pipeline import RolloutPipeline
from oracle import hts_oracle as orc
from gpu_util import rel_err

pytestmark = pytest.mark.gpu
SEED = 0xA11CE


def run_pipeline(cfg, T, N, rollouts, ring, overlap=True):
    """Runs `rollouts` rollouts; returns per scanned rollout the storage contents copied out on the scan
    stream right after its scan (values, actions, logp, adv, ret and the bootstrap row it used)."""
    dev = torch.device("cuda")
    ctx = hts.hts_policy_create(cfg.C, cfg.H, cfg.W, cfg.A, hts.HTS_DTYPE_BF16, N)
    params = wl.make_weights(cfg)
    hts.hts_policy_load_weights(ctx, hts.weights_to_device(params, hts.HTS_DTYPE_BF16))
    obs_host = [wl.make_obs(cfg, N, batch_index=i) for i in range(ring)]
    obs_dev = [torch.from_numpy(o).to(dev) for o in obs_host]
    r_np, _, d_np, _ = wl.make_rollout(cfg, T=T, N=N)
    rewards, dones = torch.from_numpy(r_np).to(dev), torch.from_numpy(d_np).to(dev)
    env_ids = torch.arange(N, dtype=torch.int32, device=dev)
    saved = {}
    pipe = None

    def after_scan(k, st):
        nxt = pipe.store[(k + 1) % 2]
        with torch.cuda.stream(pipe.s_gae):
            saved[k] = {"values": st.values.clone(), "actions": st.actions.clone(), "logp": st.logp.clone(),
                        "entropy": st.entropy.clone(), "adv": st.adv.clone(), "ret": st.ret.clone(),
                        "boot": nxt.values[0].clone()}

    pipe = RolloutPipeline(ctx, T, N, env_ids, rewards, dones, cfg.gamma, cfg.lam,
                           obs_for=lambda k, t: obs_dev[(k * T + t) % ring], seed_for=lambda k: SEED + k,
                           overlap=overlap, after_scan=after_scan)
    for k in range(rollouts):
        pipe.rollout(k)
    pipe.join()
    torch.cuda.synchronize()
    assert hts.hts_last_async_error(ctx) == 0
    hts.hts_policy_destroy(ctx)
    host = {k: {n: v.cpu().numpy() for n, v in s.items()} for k, s in saved.items()}
    return host, params, obs_host, r_np, d_np


def check_rollouts(cfg, T, N, host, params, obs_host, r_np, d_np, ring, step_samples, row_samples):
    wt = orc.Weights(params)
    for k, s in sorted(host.items()):
        # the scan: oracle on the GPU's own value rows and the bootstrap row it was given (value row 0 of k+1)
        a_ref, q_ref = orc.gae(r_np, s["values"], d_np, s["boot"], np.float32(cfg.gamma), np.float32(cfg.lam))
        assert rel_err(s["adv"], a_ref) <= 1e-5, ("adv", k)
        assert rel_err(s["ret"], q_ref) <= 1e-5, ("ret", k)
        # the same scan run again, alone, on the copied inputs: the overlapped one must give the same bits
        dev = "cuda"
        adv2 = torch.empty(T, N, device=dev); ret2 = torch.empty_like(adv2)
        hts.hts_gae(torch.from_numpy(r_np).to(dev), torch.from_numpy(s["values"]).to(dev), torch.from_numpy(d_np).to(dev),
                    torch.from_numpy(s["boot"]).to(dev), cfg.gamma, cfg.lam, T, N, adv2, ret2)
        torch.cuda.synchronize()
        assert np.array_equal(adv2.cpu().numpy().view(np.int32), s["adv"].view(np.int32))
        assert np.array_equal(ret2.cpu().numpy().view(np.int32), s["ret"].view(np.int32))
        # the actor rows that fed it: sampled steps and rows against the oracle's policy step
        g = np.random.default_rng(1000 + k)
        for t in step_samples:
            rows = np.arange(N) if N <= row_samples else np.sort(g.choice(N, row_samples, replace=False))
            ref = orc.policy_step(wt, obs_host[(k * T + t) % ring][rows], rows.astype(np.int32), t, SEED + k)
            assert rel_err(s["values"][t][rows], ref["values"]) <= 2e-2, ("values", k, t)
            sure = ref["gap"] > 0.05                     # far above any logit error of this path
            assert np.array_equal(s["actions"][t][rows][sure], ref["actions"][sure]), ("actions", k, t)
            lp_scale = max(1.0, float(np.sqrt(np.mean(ref["logits"] ** 2))))
            assert np.abs(s["logp"][t][rows][sure] - ref["logp"][sure]).max() <= 8e-2 * lp_scale


def test_overlapped_rollouts_cfg2_full_size():
    cfg = wl.CONFIGS[2]
    T, N, ring = cfg.T, cfg.N, 25
    host, params, obs_host, r_np, d_np = run_pipeline(cfg, T, N, rollouts=5, ring=ring)
    assert sorted(host) == [0, 1, 2, 3]                 # every rollout but the last has been scanned
    check_rollouts(cfg, T, N, host, params, obs_host, r_np, d_np, ring, step_samples=range(T), row_samples=64)


def test_overlapped_rollouts_T128_N1024():
    cfg = wl.CONFIGS[3]
    T, N, ring = cfg.T, cfg.N, 8
    host, params, obs_host, r_np, d_np = run_pipeline(cfg, T, N, rollouts=3, ring=ring)
    assert sorted(host) == [0, 1]
    check_rollouts(cfg, T, N, host, params, obs_host, r_np, d_np, ring, step_samples=(0, 1, 64, 127), row_samples=48)


def test_overlapped_and_serial_schedules_agree_bit_for_bit():
    cfg = wl.CONFIGS[2]
    T, N, ring = 7, 200, 14
    a, *_ = run_pipeline(cfg, T, N, rollouts=4, ring=ring, overlap=True)
    b, *_ = run_pipeline(cfg, T, N, rollouts=4, ring=ring, overlap=False)
    assert sorted(a) == sorted(b) == [0, 1, 2]
    for k in a:
        for name in a[k]:
            assert np.array_equal(a[k][name].view(np.int32), b[k][name].view(np.int32)), (k, name)
