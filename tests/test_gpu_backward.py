"""CUDA gradient of the learner objective against the CPU oracle, and one whole delayed update (Eq. 5) through
the C ABI: evaluate -> gradient -> update -> hand the new weights to the actor."""
import dataclasses

import numpy as np
import pytest
import torch

import hts_workloads as wl
import paper_2012_09849_b200 as hts
from oracle import hts_oracle as orc
from gpu_util import Policy, rel_err

pytestmark = pytest.mark.gpu
TOL = 1e-4          # fp32 arithmetic against fp64, relative with the tensor's rms as floor


def gpu_gradient(pol, obs, actions, adv, ret, logp_old, cv, ce, clip):
    n = obs.shape[0]
    dev = "cuda"
    grads = {k: torch.full(v.shape, float("nan"), dtype=torch.float32, device=dev) for k, v in pol.params.items()}
    lo = None if logp_old is None else torch.from_numpy(np.asarray(logp_old, np.float32)).to(dev)
    hts.hts_policy_gradient(pol.ctx, torch.from_numpy(obs).to(dev), torch.from_numpy(np.asarray(actions, np.int32)).to(dev),
                            torch.from_numpy(np.asarray(adv, np.float32)).to(dev),
                            torch.from_numpy(np.asarray(ret, np.float32)).to(dev), lo, cv, ce, clip, n, grads)
    torch.cuda.synchronize()
    return {k: v.cpu().numpy() for k, v in grads.items()}


def make_batch(cfg, n, seed):
    g = np.random.default_rng(seed)
    obs = wl.make_obs(cfg, n, batch_index=seed)
    actions = g.integers(0, cfg.A, n)
    adv = g.standard_normal(n).astype(np.float32)
    ret = g.standard_normal(n).astype(np.float32)
    return obs, actions, adv, ret


def check(pol, obs, actions, adv, ret, logp_old, cv, ce, clip):
    got = gpu_gradient(pol, obs, actions, adv, ret, logp_old, cv, ce, clip)
    assert hts.hts_last_async_error(pol.ctx) == 0
    f = lambda x: float(np.float32(x))
    ref = orc.objective_grad(orc.Weights(pol.params), obs, actions, adv, ret, f(cv), f(ce),
                             logp_old=logp_old, clip=f(clip))
    for k in ref:
        assert got[k].shape == ref[k].shape, k
        assert np.all(np.isfinite(got[k])), k
        e = rel_err(got[k], ref[k])
        assert e <= TOL, (k, e)
    return got, ref


@pytest.mark.parametrize("n", [16, 5])
def test_actor_critic_gradient_cfg1(n):
    cfg = wl.CONFIGS[1]
    pol = Policy(cfg, max_batch=16)
    try:
        obs, actions, adv, ret = make_batch(cfg, n, 10 + n)
        check(pol, obs, actions, adv, ret, None, 0.5, 0.01, 0.0)
    finally:
        pol.close()


def test_clipped_surrogate_gradient_both_sides_of_the_clip_range():
    cfg = wl.CONFIGS[1]
    n = 12
    pol = Policy(cfg, max_batch=n)
    try:
        obs, actions, adv, ret = make_batch(cfg, n, 3)
        ev = orc.evaluate_actions(orc.Weights(pol.params), obs, actions)
        shift = np.tile(np.array([0.4, -0.4, 0.05, -0.05]), 3)           # ratios 1.49, 0.67, 1.05, 0.95
        lo = (ev["logp"] - shift).astype(np.float32)
        got, ref = check(pol, obs, actions, adv, ret, lo, 0.5, 0.01, 0.2)
        # and a wide clip range with the ratio at one is the actor-critic gradient
        a, _ = check(pol, obs, actions, adv, ret, ev["logp"].astype(np.float32), 0.5, 0.01, 10.0)
        b, _ = check(pol, obs, actions, adv, ret, None, 0.5, 0.01, 0.0)
        for k in a:
            assert rel_err(a[k], b[k]) <= 1e-5, k
    finally:
        pol.close()


def test_full_size_batch_is_the_mean_of_its_halves():
    """At the size bench.py times (1024 samples of the cfg3 network) the oracle's backward pass is out of reach; the
    objective is a sample mean, so the gradient of a batch is the mean of the gradients of its halves, and a few
    samples of the batch alone are checked against the oracle."""
    cfg = dataclasses.replace(wl.CONFIGS[3], weight_dtype="fp32")
    n = 1024
    pol = Policy(cfg, max_batch=n)
    try:
        obs, actions, adv, ret = make_batch(cfg, n, 77)
        whole = gpu_gradient(pol, obs, actions, adv, ret, None, 0.5, 0.01, 0.0)
        h = n // 2
        lo = gpu_gradient(pol, obs[:h], actions[:h], adv[:h], ret[:h], None, 0.5, 0.01, 0.0)
        hi = gpu_gradient(pol, obs[h:], actions[h:], adv[h:], ret[h:], None, 0.5, 0.01, 0.0)
        assert hts.hts_last_async_error(pol.ctx) == 0
        for k in whole:
            assert np.all(np.isfinite(whole[k])), k
            assert rel_err(whole[k], 0.5 * (lo[k].astype(np.float64) + hi[k])) <= 1e-5, k
        rows = np.array([0, 511, 512, 1023])
        check(pol, obs[rows], actions[rows], adv[rows], ret[rows], None, 0.5, 0.01, 0.0)
    finally:
        pol.close()


@pytest.mark.parametrize("C,H,W,A,n", [(8, 44, 52, 5, 7), (4, 84, 84, 18, 33), (16, 72, 96, 19, 4)])
def test_other_shapes(C, H, W, A, n):
    cfg = dataclasses.replace(wl.CONFIGS[1], C=C, H=H, W=W, A=A)
    pol = Policy(cfg, max_batch=40)
    try:
        obs, actions, adv, ret = make_batch(cfg, n, H + n)
        check(pol, obs, actions, adv, ret, None, 0.25, 0.02, 0.0)
    finally:
        pol.close()


def test_bad_action_and_refusals():
    cfg = wl.CONFIGS[1]
    n = 6
    pol = Policy(cfg, max_batch=8)
    try:
        obs, actions, adv, ret = make_batch(cfg, n, 1)
        bad = actions.copy(); bad[2] = cfg.A                               # out of range: flagged, never an index
        got = gpu_gradient(pol, obs, bad, adv, ret, None, 0.5, 0.0, 0.0)
        assert hts.hts_last_async_error(pol.ctx) == 1
        assert all(np.all(np.isfinite(v)) for v in got.values())
        for kw in (dict(n=0), dict(n=9), dict(clip=-0.1), dict(cv=float("nan"))):
            with pytest.raises(hts.HtsError) as e:
                grads = {k: torch.zeros(v.shape, device="cuda") for k, v in pol.params.items()}
                hts.hts_policy_gradient(pol.ctx, torch.from_numpy(obs).cuda(), torch.from_numpy(actions.astype(np.int32)).cuda(),
                                        torch.from_numpy(adv).cuda(), torch.from_numpy(ret).cuda(), None,
                                        kw.get("cv", 0.5), 0.0, kw.get("clip", 0.0), kw.get("n", n), grads)
            assert e.value.status == 1
        # a tensor-core (bf16) context has no backward pass
        cfg2 = wl.CONFIGS[2]
        pol2 = Policy(cfg2, max_batch=8)
        try:
            with pytest.raises(hts.HtsError) as e:
                grads = {k: torch.zeros(v.shape, device="cuda") for k, v in pol2.params.items()}
                hts.hts_policy_gradient(pol2.ctx, torch.zeros(6, 4, 84, 84, dtype=torch.uint8, device="cuda"),
                                        torch.zeros(6, dtype=torch.int32, device="cuda"), torch.zeros(6, device="cuda"),
                                        torch.zeros(6, device="cuda"), None, 0.5, 0.0, 0.0, 6, grads)
            assert e.value.status == 6
        finally:
            pol2.close()
    finally:
        pol.close()


def test_one_delayed_update_from_rollout_to_new_actor_weights():
    """Eq. 5 end to end: the learner (fp32 master weights theta_{j-1}) takes the gradient on data collected with
    theta_{j-1}, adds it to theta_j with the RMSProp scaling of the hyper-parameter tables, and the actor (tensor-core
    context) continues with the bf16 copy of theta_{j+1}; every stage against the oracle."""
    cfg = dataclasses.replace(wl.CONFIGS[2], weight_dtype="fp32")        # learner's master copy in fp32
    n = 24
    params_prev = wl.make_weights(cfg, sub=0)                             # theta_{j-1}: behaviour = gradient point
    params_cur = wl.make_weights(cfg, sub=1)                              # theta_j: what the update is added to
    learner = Policy(cfg, params=params_prev, max_batch=n)
    actor_cfg = dataclasses.replace(cfg, weight_dtype="bf16")
    actor = None
    try:
        obs, _, _, _ = make_batch(cfg, n, 7)
        ids = np.arange(n, dtype=np.int32)
        roll = learner.step(obs, ids, 3, 99)                              # data collected with theta_{j-1}
        g = np.random.default_rng(11)
        ret = (roll["values"] + g.standard_normal(n)).astype(np.float32)
        adv = (ret - roll["values"]).astype(np.float32)
        got, ref = check(learner, obs, roll["actions"], adv, ret, None, 0.5, 0.01, 0.0)
        # the update, tensor by tensor, with a bf16 copy for the actor
        lr, alpha, eps = 7e-4, 0.99, 1e-5
        new_params, dev_bf16 = {}, {}
        for k in hts.WEIGHT_NAMES:
            theta = torch.from_numpy(params_cur[k].astype(np.float32)).cuda().contiguous()
            grad = torch.from_numpy(got[k]).cuda().contiguous()
            sq = torch.zeros_like(theta)
            half = torch.empty(theta.shape, dtype=torch.bfloat16, device="cuda")
            hts.hts_delayed_update(theta, grad, sq, theta.numel(), lr, alpha, eps, half)
            torch.cuda.synchronize()
            t_ref, _ = orc.delayed_update(params_cur[k], ref[k], np.zeros_like(params_cur[k], dtype=np.float64), lr, alpha, eps)
            # the step is lr * g / (sqrt((1-alpha) g^2) + eps): where |g| is far below eps / sqrt(1-alpha) = 1e-4 the
            # scaled step follows the relative error of g, so compare the step against its own size
            step_ref = t_ref - params_cur[k]
            step_got = theta.cpu().numpy().astype(np.float64) - params_cur[k]
            assert np.abs(step_got - step_ref).max() <= 2e-3 * max(np.abs(step_ref).max(), 1e-12) + 1e-7, k
            new_params[k] = theta.cpu().numpy()
            dev_bf16[k] = half
        actor = Policy(actor_cfg, params={k: wl.round_to_bf16(v) for k, v in new_params.items()}, max_batch=n)
        hts.hts_policy_load_weights(actor.ctx, dev_bf16)                  # hand-over of the device copy itself
        nxt = actor.step(obs, ids, 4, 99)
        ref_next = orc.policy_step(orc.Weights(actor.params), obs, ids, 4, 99)
        assert rel_err(nxt["logits"], ref_next["logits"]) <= 2e-2
        assert rel_err(nxt["values"], ref_next["values"]) <= 2e-2
        sure = ref_next["gap"] > 0.05
        assert np.array_equal(nxt["actions"][sure], ref_next["actions"][sure])
        # ascent: a small plain step along the gradient raises the objective it is the gradient of
        wt0 = orc.Weights(params_prev)
        j0 = orc.objective(wt0, obs, roll["actions"], adv, ret, 0.5, 0.01)
        stepped = {k: params_prev[k].astype(np.float64) + 1e-3 * got[k] for k in params_prev}
        j1 = orc.objective(orc.Weights(stepped), obs, roll["actions"], adv, ret, 0.5, 0.01)
        assert j1 > j0
    finally:
        learner.close()
        if actor is not None:
            actor.close()
