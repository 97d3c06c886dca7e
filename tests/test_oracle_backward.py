"""Pins of the oracle's gradient of the learner objective (the quantity Eq. 4 estimates): central differences on
the forward oracle, a library autograd in fp64, and cases with a closed form."""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

import hts_workloads as wl
from oracle import hts_oracle as orc

CFG = wl.CONFIGS[1]


def _case(n=3, seed=0, small=True):
    """A small frame (so that finite differences over the forward oracle stay cheap) with the paper's layers."""
    import dataclasses
    cfg = dataclasses.replace(CFG, H=44, W=52, A=5) if small else CFG
    params = wl.make_weights(cfg, sub=seed)
    g = np.random.default_rng(seed)
    obs = wl.make_obs(cfg, n, batch_index=seed)
    actions = g.integers(0, cfg.A, n)
    adv = g.standard_normal(n)
    ret = g.standard_normal(n)
    logp_old = -np.abs(g.standard_normal(n)) - 0.5
    return cfg, params, obs, actions, adv, ret, logp_old


def _torch_objective(params, obs, actions, adv, ret, cv, ce, logp_old=None, clip=0.0):
    t = {k: torch.tensor(v, dtype=torch.float64, requires_grad=True) for k, v in params.items()}
    x = torch.tensor(obs.astype(np.float64) / 255.0)
    y = F.relu(F.conv2d(x, t["conv1_w"], t["conv1_b"], stride=4))
    y = F.relu(F.conv2d(y, t["conv2_w"], t["conv2_b"], stride=2))
    y = F.relu(F.conv2d(y, t["conv3_w"], t["conv3_b"], stride=1))
    h = F.relu(F.linear(y.flatten(1), t["fc_w"], t["fc_b"]))
    logits = F.linear(h, t["pi_w"], t["pi_b"])
    value = F.linear(h, t["v_w"], t["v_b"])[:, 0]
    logp = F.log_softmax(logits, dim=1)
    ent = -(logp.exp() * logp).sum(dim=1)
    lpa = logp[torch.arange(len(actions)), torch.tensor(actions)]
    A, R = torch.tensor(adv), torch.tensor(ret)
    if logp_old is None or clip <= 0:
        s = lpa * A
    else:
        rho = (lpa - torch.tensor(logp_old)).exp()
        s = torch.minimum(rho * A, rho.clamp(1 - clip, 1 + clip) * A)
    J = (s - cv * (R - value) ** 2 + ce * ent).mean()
    J.backward()
    return float(J), {k: v.grad.numpy() for k, v in t.items()}


@pytest.mark.parametrize("mode", ["a2c", "ppo"])
def test_gradient_equals_library_autograd(mode):
    cfg, params, obs, actions, adv, ret, lo = _case(n=4, seed=1)
    wt = orc.Weights(params)
    kw = dict(logp_old=lo + 1.2, clip=0.2) if mode == "ppo" else {}
    if mode == "ppo":                                   # put the ratios on both sides of the clip range
        ev = orc.evaluate_actions(wt, obs, actions)
        kw["logp_old"] = ev["logp"] - np.array([0.3, -0.3, 0.05, -0.05])
    g = orc.objective_grad(wt, obs, actions, adv, ret, 0.5, 0.01, **kw)
    J, gt = _torch_objective(params, obs, actions, adv, ret, 0.5, 0.01, **kw)
    assert abs(J - orc.objective(wt, obs, actions, adv, ret, 0.5, 0.01, **kw)) < 1e-12
    for k in gt:
        assert g[k].shape == gt[k].shape, k
        scale = max(np.abs(gt[k]).max(), 1e-30)
        assert np.abs(g[k] - gt[k]).max() <= 1e-10 * scale, k


def test_gradient_equals_central_differences_of_the_forward_oracle():
    cfg, params, obs, actions, adv, ret, _ = _case(n=2, seed=2)
    wt = orc.Weights(params)
    g = orc.objective_grad(wt, obs, actions, adv, ret, 0.5, 0.02)
    rng = np.random.default_rng(3)
    eps = 1e-5
    for name in orc.Weights.NAMES:
        flat = params[name].reshape(-1)
        for idx in rng.choice(flat.size, size=min(3, flat.size), replace=False):
            vals = []
            for sgn in (+1, -1):
                p2 = {k: v.astype(np.float64).copy() for k, v in params.items()}
                p2[name].reshape(-1)[idx] += sgn * eps
                vals.append(orc.objective(orc.Weights(p2), obs, actions, adv, ret, 0.5, 0.02))
            fd = (vals[0] - vals[1]) / (2 * eps)
            an = g[name].reshape(-1)[idx]
            assert abs(fd - an) <= 1e-6 * max(1.0, abs(an)) + 1e-8, (name, idx, fd, an)


def test_closed_form_cases():
    cfg, params, obs, actions, adv, ret, _ = _case(n=3, seed=4)
    wt = orc.Weights(params)
    # no advantage, no entropy bonus: only the value loss speaks; the policy head gets no gradient
    g = orc.objective_grad(wt, obs, actions, np.zeros(3), ret, 0.5, 0.0)
    assert np.all(g["pi_w"] == 0) and np.all(g["pi_b"] == 0) and np.any(g["v_w"] != 0)
    ev = orc.evaluate_actions(wt, obs, actions)
    assert np.allclose(g["v_b"], [np.mean(2 * 0.5 * (ret - ev["values"]))], rtol=1e-12)
    # returns equal to the values and no entropy bonus: the value head gets none, the policy bias gradient is the
    # mean of A_i (onehot(a_i) - pi_i)
    g = orc.objective_grad(wt, obs, actions, adv, ev["values"], 0.5, 0.0)
    assert np.all(g["v_w"] == 0) and np.all(g["v_b"] == 0)
    p = np.exp(ev["logits"] - ev["logits"].max(1, keepdims=True)); p /= p.sum(1, keepdims=True)
    onehot = np.eye(cfg.A)[actions]
    assert np.allclose(g["pi_b"], (adv[:, None] * (onehot - p)).mean(0), rtol=1e-10, atol=1e-14)
    # PPO with the ratio at one and a wide clip range is the actor-critic gradient
    g1 = orc.objective_grad(wt, obs, actions, adv, ret, 0.5, 0.01)
    g2 = orc.objective_grad(wt, obs, actions, adv, ret, 0.5, 0.01, logp_old=ev["logp"], clip=0.2)
    for k in g1:
        assert np.abs(g1[k] - g2[k]).max() <= 1e-12 * max(np.abs(g1[k]).max(), 1e-300), k
    # a ratio clipped on the side the advantage pushes towards contributes no policy gradient
    g3 = orc.objective_grad(wt, obs, actions, np.abs(adv), ev["values"], 0.5, 0.0, logp_old=ev["logp"] - 1.0, clip=0.2)
    assert np.all(g3["pi_b"] == 0) and np.all(g3["conv1_w"] == 0)
    # linearity in the advantages (entropy and value terms off)
    ga = orc.objective_grad(wt, obs, actions, adv, ev["values"], 0.0, 0.0)
    gb = orc.objective_grad(wt, obs, actions, 3.0 * adv, ev["values"], 0.0, 0.0)
    for k in ga:
        assert np.abs(3.0 * ga[k] - gb[k]).max() <= 1e-12 * max(np.abs(gb[k]).max(), 1e-300), k
