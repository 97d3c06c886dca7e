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
