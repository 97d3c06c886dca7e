"""Learner-side entry points against the oracle: hts_policy_evaluate (re-evaluation of stored actions) and
hts_a2c_terms (the sample means of Eq. 4 and of the value loss)."""
import os

import numpy as np
import pytest
import torch

import hts_workloads as wl
import paper_2012_09849_b200 as hts
from oracle import hts_oracle as orc
from gpu_util import Policy, rel_err

pytestmark = pytest.mark.gpu
GOLD = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "a2c_terms_worked_example.txt")


def evaluate(pol, obs, actions, want_logits=True):
    n = obs.shape[0]
    d_obs = torch.from_numpy(np.ascontiguousarray(obs)).cuda()
    d_act = torch.from_numpy(np.ascontiguousarray(actions, dtype=np.int32)).cuda()
    logp, val, ent = (torch.full((n,), -9.0, dtype=torch.float32, device="cuda") for _ in range(3))
    logits = torch.empty(n, pol.cfg.A, dtype=torch.float32, device="cuda") if want_logits else None
    hts.hts_policy_evaluate(pol.ctx, d_obs, d_act, n, logp, val, ent, logits)
    torch.cuda.synchronize()
    out = {"logp": logp.cpu().numpy(), "values": val.cpu().numpy(), "entropy": ent.cpu().numpy()}
    if want_logits:
        out["logits"] = logits.cpu().numpy()
    return out


@pytest.mark.parametrize("ci,n", [(1, 16), (2, 150), (4, 40)])
def test_evaluate_matches_oracle_and_the_actor_step(ci, n):
    cfg = wl.CONFIGS[ci]
    pol = Policy(cfg, max_batch=n)
    try:
        g = np.random.default_rng(ci)
        obs = wl.make_obs(cfg, n, batch_index=21)
        actions = g.integers(0, cfg.A, n).astype(np.int32)            # arbitrary stored actions
        got = evaluate(pol, obs, actions)
        assert hts.hts_last_async_error(pol.ctx) == 0
        rows = np.arange(n) if n <= 48 else np.sort(g.choice(n, 48, replace=False))
        ref = orc.evaluate_actions(orc.Weights(pol.params), obs[rows], actions[rows])
        tol = 1e-4 if cfg.weight_dtype == "fp32" else 2e-2
        scale = max(1.0, float(np.sqrt(np.mean(ref["logits"] ** 2))))
        assert rel_err(got["logits"][rows], ref["logits"]) <= tol
        assert rel_err(got["values"][rows], ref["values"]) <= tol
        assert np.abs(got["logp"][rows] - ref["logp"]).max() <= 4 * tol * scale
        assert np.abs(got["entropy"][rows] - ref["entropy"]).max() <= 4 * tol * scale
        # given the GPU's own logits, log-prob and entropy are the oracle's to fp32 rounding
        for e in rows[:16]:
            lp, h = orc.log_softmax(got["logits"][e].astype(np.float64))
            assert abs(got["logp"][e] - lp[actions[e]]) <= 2e-5 * max(1.0, abs(lp[actions[e]]))
            assert abs(got["entropy"][e] - h) <= 2e-5 * max(1.0, h)
        # the action the actor sampled, re-evaluated: the step's own numbers, bit for bit
        step = pol.step(obs, np.arange(n), 7, 31, want_logits=False)
        again = evaluate(pol, obs, step["actions"], want_logits=False)
        for k in ("logp", "values", "entropy"):
            assert np.array_equal(again[k], step[k]), k
    finally:
        pol.close()


def test_evaluate_reports_an_action_outside_the_range():
    cfg = wl.CONFIGS[2]
    n = 6
    pol = Policy(cfg, max_batch=n)
    try:
        obs = wl.make_obs(cfg, n, batch_index=2)
        actions = np.array([0, cfg.A, 3, -1, cfg.A - 1, 1], dtype=np.int32)
        got = evaluate(pol, obs, actions, want_logits=False)
        assert hts.hts_last_async_error(pol.ctx) == 1 and hts.hts_last_async_error(pol.ctx) == 0
        bad = (actions < 0) | (actions >= cfg.A)
        assert np.all(got["logp"][bad] == -9.0) and np.all(got["logp"][~bad] != -9.0)
        L = hts.lib()
        assert L.hts_policy_evaluate(pol.ctx, 8, None, n, 16, 24, 32, None, None) == 1
        assert L.hts_policy_evaluate(pol.ctx, 8, 16, n + 1, 24, 32, 40, None, None) == 1
    finally:
        pol.close()


def gpu_terms(logp, v, h, r):
    t = [torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda() for a in (logp, v, h, r)]
    out = torch.zeros(3, dtype=torch.float32, device="cuda")
    hts.hts_a2c_terms(*t, t[0].numel(), out)
    torch.cuda.synchronize()
    return out.cpu().numpy()


def test_a2c_terms_worked_example_on_gpu():
    rows, expected = [], None
    for line in open(GOLD, encoding="utf-8"):
        line = line.strip()
        if line.startswith("expected"):
            expected = [float(x) for x in line.split()[1:]]
        elif line and not line.startswith("#"):
            rows.append([float(x) for x in line.split()])
    a = np.array(rows)
    assert list(gpu_terms(a[:, 0], a[:, 1], a[:, 2], a[:, 3])) == expected


@pytest.mark.parametrize("count", [1, 3, 4, 5, 1023, 8192, 8193, 131072, 1 << 22, (1 << 22) + 7, 12345677])
def test_a2c_terms_against_oracle(count):
    g = np.random.default_rng(count)
    logp = -g.random(count, dtype=np.float32) * 3
    v, r = g.standard_normal(count, dtype=np.float32), g.standard_normal(count, dtype=np.float32)
    h = g.random(count, dtype=np.float32) * 2.8
    got = gpu_terms(logp, v, h, r)
    if count <= 200000:
        ref = np.array(orc.a2c_terms(logp, v, h, r))
    else:                                               # the definition through fp64 library reductions at size
        a = r.astype(np.float64) - v
        ref = np.array([np.mean(logp * a), np.mean(a * a), np.mean(h, dtype=np.float64)])
    floor = np.array([np.sqrt(np.mean((logp.astype(np.float64) * (r.astype(np.float64) - v)) ** 2)) / np.sqrt(count), 1.0, 1.0])
    assert np.all(np.abs(got - ref) <= 1e-6 * np.maximum(np.abs(ref), floor)), (got, ref)
    assert np.array_equal(got, gpu_terms(logp, v, h, r))                # same bits on a second run


def test_a2c_terms_unaligned_views_and_refusals():
    g = np.random.default_rng(1)
    n = 5001
    base = [torch.from_numpy(g.standard_normal(n + 3, dtype=np.float32)).cuda() for _ in range(4)]
    views = [b[1:n + 1] for b in base]                                  # 4-byte aligned only
    out = torch.zeros(3, dtype=torch.float32, device="cuda")
    hts.hts_a2c_terms(*views, n, out)
    torch.cuda.synchronize()
    ref = np.array(orc.a2c_terms(*[v.cpu().numpy() for v in views]))
    assert np.all(np.abs(out.cpu().numpy() - ref) <= 1e-6 * np.maximum(np.abs(ref), 1e-2))
    L = hts.lib()
    assert L.hts_a2c_terms(8, 16, 24, 32, 0, 40, None) == 1
    assert L.hts_a2c_terms(None, 16, 24, 32, 4, 40, None) == 1


@pytest.mark.parametrize("count", [1, 5, 1025, 1693875, (1 << 22) + 3])
def test_delayed_update_against_oracle(count):
    g = np.random.default_rng(count)
    theta = g.standard_normal(count, dtype=np.float32)
    grad = (g.standard_normal(count, dtype=np.float32) * 0.1).astype(np.float32)
    v = (g.random(count, dtype=np.float32) * 0.01).astype(np.float32)
    lr, alpha, eps = np.float32(7e-4), np.float32(0.99), np.float32(1e-5)
    d_t, d_g, d_v = (torch.from_numpy(a.copy()).cuda() for a in (theta, grad, v))
    d_b = torch.empty(count, dtype=torch.bfloat16, device="cuda")
    hts.hts_delayed_update(d_t, d_g, d_v, count, lr, alpha, eps, d_b)
    torch.cuda.synchronize()
    n_ref = min(count, 20000)                                   # the oracle is a Python loop
    rt, rv = orc.delayed_update(theta[:n_ref], grad[:n_ref], v[:n_ref], float(lr), float(alpha), float(eps))
    got_t, got_v = d_t.cpu().numpy(), d_v.cpu().numpy()
    assert np.all(np.abs(got_v[:n_ref] - rv) <= 1e-6 * np.maximum(np.abs(rv), 1e-8))
    assert np.all(np.abs(got_t[:n_ref] - rt) <= 1e-6 * np.maximum(np.abs(rt), 1e-3))
    # at size: the rule through fp64 library expressions
    vv = float(alpha) * v.astype(np.float64) + (1.0 - float(alpha)) * grad.astype(np.float64) ** 2
    tt = theta + float(lr) * grad / (np.sqrt(vv) + float(eps))
    assert np.all(np.abs(got_t - tt) <= 1e-6 * np.maximum(np.abs(tt), 1e-3))
    # the bf16 copy is the new fp32 parameter rounded to nearest even
    assert torch.equal(d_b, d_t.to(torch.bfloat16))
    # plain Eq. 5
    d_t2 = torch.from_numpy(theta.copy()).cuda()
    hts.hts_delayed_update(d_t2, d_g, None, count, 0.5, 0.0, 0.0)
    torch.cuda.synchronize()
    scale = np.maximum(np.maximum(np.abs(theta), np.abs(0.5 * grad)), 1e-3)         # fp32 rounding of the larger operand
    assert np.all(np.abs(d_t2.cpu().numpy() - (theta + 0.5 * grad.astype(np.float64))) <= 1e-6 * scale)


def test_delayed_update_golden_and_refusals():
    path = os.path.join(os.path.dirname(GOLD), "delayed_update_worked_example.txt")
    rows, exp = [], {}
    for line in open(path, encoding="utf-8"):
        line = line.split("#")[0].strip()
        if line.startswith("expected"):
            k, *vals = line.split()
            exp[k] = np.array([float(x) for x in vals])
        elif line:
            rows.append([float(x) for x in line.split()])
    a = np.array(rows, dtype=np.float32)
    d_t, d_g, d_v = (torch.from_numpy(a[:, i].copy()).cuda() for i in range(3))
    hts.hts_delayed_update(d_t, d_g, d_v, 4, 0.5, 0.75, 0.5)
    torch.cuda.synchronize()
    assert np.array_equal(d_v.cpu().numpy(), exp["expected_v"].astype(np.float32))
    assert np.allclose(d_t.cpu().numpy(), exp["expected_theta"], rtol=2e-7, atol=0)
    # views that are only 4-byte aligned take the scalar path and give the same numbers
    g = np.random.default_rng(2)
    n = 1003
    base = [torch.from_numpy(g.standard_normal(n + 1, dtype=np.float32)).abs().cuda() for _ in range(3)]
    al = [b[:n].clone() for b in base]
    un = [b.clone()[1:] for b in [torch.cat([b[:1], b[:n]]) for b in base]]
    hts.hts_delayed_update(al[0], al[1], al[2], n, 0.01, 0.9, 1e-3)
    hts.hts_delayed_update(un[0], un[1], un[2], n, 0.01, 0.9, 1e-3)
    torch.cuda.synchronize()
    assert torch.equal(al[0], un[0]) and torch.equal(al[2], un[2])
    L = hts.lib()
    assert L.hts_delayed_update(None, 8, 16, 4, 0.1, 0.9, 1e-5, None, None) == 1
    assert L.hts_delayed_update(8, 16, 24, 0, 0.1, 0.9, 1e-5, None, None) == 1
    assert L.hts_delayed_update(8, 16, 24, 4, 0.1, 1.5, 1e-5, None, None) == 1
    assert L.hts_delayed_update(8, 16, 24, 4, 0.1, 0.9, 0.0, None, None) == 1
    assert L.hts_delayed_update(8, 16, 24, 4, float("nan"), 0.9, 1e-5, None, None) == 1


def gpu_ppo(ln, lo, v, h, a, r, clip, normalize):
    t = [torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).cuda() for x in (ln, lo, v, h, a, r)]
    out = torch.zeros(4, dtype=torch.float32, device="cuda")
    hts.hts_ppo_terms(*t, t[0].numel(), clip, normalize, out)
    torch.cuda.synchronize()
    return out.cpu().numpy()


def test_ppo_terms_worked_example_on_gpu():
    path = os.path.join(os.path.dirname(GOLD), "ppo_terms_worked_example.txt")
    rows, exp = [], None
    for line in open(path, encoding="utf-8"):
        line = line.split("#")[0].strip()
        if line.startswith("expected"):
            exp = np.array([float(x) for x in line.split()[1:]])
        elif line:
            rows.append([float(x) for x in line.split()])
    a = np.array(rows)
    lo = np.full(len(a), -1.5, dtype=np.float32)
    ln = (lo.astype(np.float64) + np.log(a[:, 0])).astype(np.float32)
    got = gpu_ppo(ln, lo, a[:, 2], a[:, 4], a[:, 1], a[:, 3], 0.25, False)
    assert np.allclose(got, exp, rtol=2e-6, atol=0)


@pytest.mark.parametrize("count,normalize", [(1, False), (7, True), (4097, False), (4097, True), (131072, True),
                                             ((1 << 21) + 5, True), (3000001, False)])
def test_ppo_terms_against_oracle(count, normalize):
    g = np.random.default_rng(count + int(normalize))
    lo = (-g.random(count, dtype=np.float32) * 3).astype(np.float32)
    ln = (lo + 0.25 * g.standard_normal(count, dtype=np.float32)).astype(np.float32)
    v, r = g.standard_normal(count, dtype=np.float32), g.standard_normal(count, dtype=np.float32)
    h = g.random(count, dtype=np.float32) * 2.8
    adv = (1.5 * g.standard_normal(count, dtype=np.float32) + 0.7).astype(np.float32)
    if count == 1:
        normalize = False
    got = gpu_ppo(ln, lo, v, h, adv, r, 0.2, normalize)
    if count <= 200000:
        ref = np.array(orc.ppo_terms(ln, lo, v, h, adv, r, 0.2, normalize))
    else:                                               # the definition through fp64 library expressions at size
        a64 = adv.astype(np.float64)
        if normalize:
            a64 = (a64 - a64.mean()) / (a64.std() + 1e-8)
        rho = np.exp(ln.astype(np.float64) - lo)
        ref = np.array([np.mean(np.minimum(rho * a64, np.clip(rho, 0.8, 1.2) * a64)),
                        np.mean((r.astype(np.float64) - v) ** 2), np.mean(h, dtype=np.float64),
                        np.mean(np.abs(rho - 1.0) > 0.2)])
    floor = np.array([1.0 / np.sqrt(count), 1.0, 1.0, 1e-3])
    # a sample whose |rho - 1| sits within rounding of the clip may fall on either side: one count of slack there
    tol = 1e-6 * np.maximum(np.abs(ref), floor) + np.array([0, 0, 0, 2.0 / count])
    assert np.all(np.abs(got - ref) <= tol), (got, ref)
    assert np.array_equal(got, gpu_ppo(ln, lo, v, h, adv, r, 0.2, normalize))


def test_ppo_terms_refusals_and_interleaving_with_a2c_terms():
    L = hts.lib()
    assert L.hts_ppo_terms(8, 16, 24, 32, 40, 48, 0, 0.2, 0, 56, None) == 1
    assert L.hts_ppo_terms(8, 16, 24, 32, 40, 48, 4, 0.0, 0, 56, None) == 1
    assert L.hts_ppo_terms(None, 16, 24, 32, 40, 48, 4, 0.2, 0, 56, None) == 1
    # the two reductions share the library's partial table: back-to-back calls on one stream must not disturb each other
    g = np.random.default_rng(0)
    n = 50001
    arrs = [g.standard_normal(n, dtype=np.float32) for _ in range(6)]
    p1 = gpu_ppo(*arrs, 0.2, True)
    a1 = gpu_terms(arrs[0], arrs[2], arrs[3], arrs[5])
    assert np.array_equal(p1, gpu_ppo(*arrs, 0.2, True)) and np.array_equal(a1, gpu_terms(arrs[0], arrs[2], arrs[3], arrs[5]))
