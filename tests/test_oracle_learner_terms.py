"""Pins of the oracle's learner-side functions (re-evaluation of stored actions, Eq. 4 sample means)."""
import os

import numpy as np
import pytest

import hts_workloads as wl
from oracle import hts_oracle as orc

GOLD = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "a2c_terms_worked_example.txt")


def test_a2c_terms_worked_example():
    rows, expected = [], None
    for line in open(GOLD, encoding="utf-8"):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        if line.startswith("expected"):
            expected = [float(x) for x in line.split()[1:]]
        else:
            rows.append([float(x) for x in line.split()])
    a = np.array(rows)
    got = orc.a2c_terms(a[:, 0], a[:, 1], a[:, 2], a[:, 3])
    assert list(got) == expected


def test_a2c_terms_closed_forms_and_invariants():
    g = np.random.default_rng(3)
    n = 257
    logp, v, h, r = -g.random(n), g.standard_normal(n), g.random(n), g.standard_normal(n)
    pol, vl, ent = orc.a2c_terms(logp, v, h, r)
    # definitions through library reductions
    assert pol == pytest.approx(float(np.mean(logp * (r - v))), rel=1e-13)
    assert vl == pytest.approx(float(np.mean((r - v) ** 2)), rel=1e-13)
    assert ent == pytest.approx(float(np.mean(h)), rel=1e-13)
    # R = V: no policy term, no value loss
    p0, v0, _ = orc.a2c_terms(logp, v, h, v)
    assert p0 == 0.0 and v0 == 0.0
    # uniform policy over A actions: policy term = -ln A * mean advantage
    A = 18
    p1, _, _ = orc.a2c_terms(np.full(n, -np.log(A)), v, h, r)
    assert p1 == pytest.approx(-np.log(A) * float(np.mean(r - v)), rel=1e-12)
    # order of the transitions does not matter; the advantage enters linearly / quadratically
    perm = g.permutation(n)
    assert orc.a2c_terms(logp[perm], v[perm], h[perm], r[perm]) == pytest.approx((pol, vl, ent), rel=1e-12)
    p2, v2, _ = orc.a2c_terms(logp, 2 * v, h, 2 * r)
    assert p2 == pytest.approx(2 * pol, rel=1e-12) and v2 == pytest.approx(4 * vl, rel=1e-12)
    # swapping the sign of the advantage flips the policy term only
    p3, v3, _ = orc.a2c_terms(logp, r, h, v)
    assert p3 == pytest.approx(-pol, rel=1e-12) and v3 == pytest.approx(vl, rel=1e-12)


def test_evaluate_actions_is_the_distribution_of_the_actor_step():
    cfg = wl.CONFIGS[1]
    wt = orc.Weights(wl.make_weights(cfg))
    n = 6
    obs = wl.make_obs(cfg, n, batch_index=4)
    ids = np.arange(n, dtype=np.int32)
    step = orc.policy_step(wt, obs, ids, 3, 99)
    ev = orc.evaluate_actions(wt, obs, step["actions"])
    # the sampled action's log-probability, the value and the entropy are those the actor reported
    assert np.allclose(ev["logp"], step["logp"], rtol=0, atol=1e-12)
    assert np.allclose(ev["values"], step["values"], rtol=0, atol=1e-12)
    assert np.allclose(ev["entropy"], step["entropy"], rtol=0, atol=1e-12)
    # over all actions the probabilities sum to one and reproduce the entropy
    for e in range(n):
        lps = np.array([orc.evaluate_actions(wt, obs[e:e + 1], [a])["logp"][0] for a in range(cfg.A)])
        assert abs(np.exp(lps).sum() - 1.0) < 1e-12
        assert abs(-(np.exp(lps) * lps).sum() - ev["entropy"][e]) < 1e-12
    with pytest.raises(AssertionError):
        orc.evaluate_actions(wt, obs, np.full(n, cfg.A))


def _gold_update():
    path = os.path.join(os.path.dirname(GOLD), "delayed_update_worked_example.txt")
    rows, exp = [], {}
    for line in open(path, encoding="utf-8"):
        line = line.split("#")[0].strip()
        if not line:
            continue
        if line.startswith("expected"):
            k, *v = line.split()
            exp[k] = np.array([float(x) for x in v])
        else:
            rows.append([float(x) for x in line.split()])
    return np.array(rows), exp


def test_delayed_update_worked_example():
    a, exp = _gold_update()
    t, v = orc.delayed_update(a[:, 0], a[:, 1], a[:, 2], lr=0.5, alpha=0.75, eps=0.5)
    assert np.array_equal(v, exp["expected_v"])
    assert np.allclose(t, exp["expected_theta"], rtol=0, atol=1e-16)
    t2, v2 = orc.delayed_update(a[:, 0], a[:, 1], a[:, 2], lr=0.5, alpha=0.75, eps=0.5, precondition=False)
    assert np.array_equal(t2, exp["expected_plain"]) and np.array_equal(v2, a[:, 2])


def test_delayed_update_closed_forms():
    g = np.random.default_rng(11)
    n = 300
    theta, grad, v = g.standard_normal(n), g.standard_normal(n), g.random(n)
    # zero gradient: parameters stay, the running average decays by alpha
    t0, v0 = orc.delayed_update(theta, np.zeros(n), v, 0.1, 0.9, 1e-5)
    assert np.array_equal(t0, theta) and np.allclose(v0, 0.9 * v, rtol=1e-15)
    # alpha = 0: v' = g^2, so the step is eta * g / (|g| + eps), bounded by eta and of the gradient's sign
    t1, v1 = orc.delayed_update(theta, grad, v, 0.1, 0.0, 1e-5)
    assert np.allclose(v1, grad ** 2, rtol=1e-15)
    assert np.allclose(t1 - theta, 0.1 * grad / (np.abs(grad) + 1e-5), rtol=1e-12)
    assert np.all(np.abs(t1 - theta) < 0.1) and np.all(np.sign(t1 - theta) == np.sign(grad))
    # library expression of the rule; ascent direction (Eq. 5 adds the gradient of the objective)
    t2, v2 = orc.delayed_update(theta, grad, v, 0.01, 0.99, 0.01)
    vv = 0.99 * v + 0.01 * grad ** 2
    assert np.allclose(v2, vv, rtol=1e-15) and np.allclose(t2, theta + 0.01 * grad / (np.sqrt(vv) + 0.01), rtol=1e-13)
    # constant gradient: v converges to g^2 and the step to eta * g / (|g| + eps)
    tt, vv = theta.copy(), np.zeros(n)
    for _ in range(2000):
        prev = tt
        tt, vv = orc.delayed_update(tt, grad, vv, 0.001, 0.99, 1e-3)
    assert np.allclose(vv, grad ** 2, rtol=1e-6)
    assert np.allclose(tt - prev, 0.001 * grad / (np.abs(grad) + 1e-3), rtol=1e-6)
    # plain Eq. 5 is linear in the gradient
    ta, _ = orc.delayed_update(theta, grad, v, 0.3, 0.9, 1e-5, precondition=False)
    tb, _ = orc.delayed_update(theta, 2 * grad, v, 0.3, 0.9, 1e-5, precondition=False)
    assert np.allclose(tb - theta, 2 * (ta - theta), rtol=1e-13)


def _gold_ppo():
    path = os.path.join(os.path.dirname(GOLD), "ppo_terms_worked_example.txt")
    rows, exp = [], None
    for line in open(path, encoding="utf-8"):
        line = line.split("#")[0].strip()
        if not line:
            continue
        if line.startswith("expected"):
            exp = [float(x) for x in line.split()[1:]]
        else:
            rows.append([float(x) for x in line.split()])
    return np.array(rows), exp


def test_ppo_terms_worked_example():
    a, exp = _gold_ppo()
    lp_old = np.full(len(a), -1.5)
    got = orc.ppo_terms(lp_old + np.log(a[:, 0]), lp_old, a[:, 2], a[:, 4], a[:, 1], a[:, 3], 0.25, False)
    assert np.allclose(got, exp, rtol=1e-15, atol=0)


def test_ppo_terms_closed_forms():
    g = np.random.default_rng(8)
    n = 400
    lo = -g.random(n) * 2
    v, r, h, adv = g.standard_normal(n), g.standard_normal(n), g.random(n), g.standard_normal(n)
    # identical policies: rho = 1, the surrogate is the mean advantage and nothing is clipped
    s, vl, ent, frac = orc.ppo_terms(lo, lo, v, h, adv, r, 0.2, False)
    assert s == pytest.approx(float(np.mean(adv)), rel=1e-13) and frac == 0.0
    assert vl == pytest.approx(float(np.mean((r - v) ** 2)), rel=1e-13) and ent == pytest.approx(float(np.mean(h)), rel=1e-13)
    # standardised advantages have mean 0: with rho = 1 the surrogate vanishes; the standardisation is shift/scale free
    s0, *_ = orc.ppo_terms(lo, lo, v, h, adv, r, 0.2, True)
    assert abs(s0) < 1e-12
    ln = lo + 0.3 * g.standard_normal(n)
    a1 = orc.ppo_terms(ln, lo, v, h, adv, r, 0.2, True)
    a2 = orc.ppo_terms(ln, lo, v, h, 5.0 * adv + 3.0, r, 0.2, True)
    assert np.allclose(a1, a2, rtol=1e-7)
    # the surrogate never exceeds the unclipped importance-weighted mean, and equals it for a huge clip range
    rho = np.exp(ln - lo)
    s1, _, _, f1 = orc.ppo_terms(ln, lo, v, h, adv, r, 0.2, False)
    assert s1 <= float(np.mean(rho * adv)) + 1e-15 and 0.0 < f1 < 1.0
    assert f1 == pytest.approx(float(np.mean(np.abs(rho - 1.0) > 0.2)), rel=1e-15)
    s2, _, _, f2 = orc.ppo_terms(ln, lo, v, h, adv, r, 1e6, False)
    assert s2 == pytest.approx(float(np.mean(rho * adv)), rel=1e-13) and f2 == 0.0
    # library expression
    ref = float(np.mean(np.minimum(rho * adv, np.clip(rho, 0.8, 1.2) * adv)))
    assert s1 == pytest.approx(ref, rel=1e-13)
