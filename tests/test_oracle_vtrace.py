"""Pins of the oracle's V-trace / truncated-importance-sampling scan: the definition of the cited paper written
out as an explicit sum, a hand-worked example, and the cases in which it reduces to the advantage scan."""
import os

import numpy as np

import hts_workloads as wl
from oracle import hts_oracle as orc

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "vtrace_worked_example.txt")


def _inputs(T=9, N=7, seed=0, p_done=0.2):
    g = np.random.default_rng(seed)
    lr = g.normal(0, 0.7, (T, N)).astype(np.float32)
    r = g.integers(-1, 2, (T, N)).astype(np.float32)
    v = g.standard_normal((T, N)).astype(np.float32)
    d = (g.random((T, N)) < p_done).astype(np.uint8)
    b = g.standard_normal(N).astype(np.float32)
    return lr, r, v, d, b


def _definition(lr, r, v, d, b, gamma, lam, rho_bar, c_bar):
    """v_s = V_s + sum_{t >= s} (prod_{i=s}^{t-1} g_i c_i) delta_t, written as the double sum it is (no recursion)."""
    T, N = r.shape
    lr, r, v, b = (np.asarray(a, np.float64) for a in (lr, r, v, b))
    ratio = np.exp(lr)
    rho, c = np.minimum(rho_bar, ratio), lam * np.minimum(c_bar, ratio)
    g = gamma * (1.0 - (np.asarray(d) != 0))
    vnext = np.vstack([v[1:], b[None]])
    delta = rho * (r + g * vnext - v)
    vs = np.empty((T, N))
    for s in range(T):
        acc = np.zeros(N)
        for t in range(s, T):
            w = np.ones(N)
            for i in range(s, t):
                w = w * g[i] * c[i]
            acc += w * delta[t]
        vs[s] = v[s] + acc
    vs_next = np.vstack([vs[1:], b[None]])
    pg = rho * (r + g * vs_next - v)
    return vs, pg


def test_recursion_equals_the_explicit_sum():
    for seed, (gamma, lam, rb, cb) in enumerate([(0.99, 1.0, 1.0, 1.0), (0.9, 0.95, 2.0, 0.7), (0.5, 1.0, 0.3, 3.0)]):
        args = _inputs(seed=seed)
        vs, pg = orc.vtrace(*args, gamma, lam, rb, cb)
        vs_d, pg_d = _definition(*args, gamma, lam, rb, cb)
        assert np.allclose(vs, vs_d, rtol=1e-6, atol=1e-6) and np.allclose(pg, pg_d, rtol=1e-6, atol=1e-6)


def test_hand_worked_example():
    text = [l.split() for l in open(GOLDEN) if l.strip() and not l.startswith("#")]
    cases, name = {}, None
    for row in text:
        if row[0] == "case":
            name = row[1]; cases[name] = {}
        else:
            cases[name][row[0]] = np.array([float(x) for x in row[1:]])
    lr = np.log(np.array([[2.0], [0.5], [1.0]]))
    r = np.array([[1.0], [0.0], [2.0]]); v = np.array([[0.5], [1.0], [0.0]]); b = np.array([4.0])
    for cname, dn in (("no_dones", [0, 0, 0]), ("done_at_1", [0, 1, 0])):
        vs, pg = orc.vtrace(lr, r, v, np.array(dn, np.uint8)[:, None], b, 0.5, 1.0, 1.0, 1.0)
        assert np.array_equal(vs[:, 0].astype(np.float64), cases[cname]["vs"]), cname
        assert np.array_equal(pg[:, 0].astype(np.float64), cases[cname]["pg"]), cname


def test_on_policy_untruncated_is_the_n_step_return():
    # pi = mu and rho_bar, c_bar >= 1: vs is the lambda = 1 return of the advantage scan, pg its advantage
    cfg = wl.CONFIGS[3]
    r, v, d, b = wl.make_rollout(cfg, T=33, N=41)
    zero = np.zeros_like(r)
    vs, pg = orc.vtrace(zero, r, v, d, b, cfg.gamma, 1.0, 1.0, 1.0)
    adv, ret = orc.gae(r, v, d, b, np.float32(cfg.gamma), np.float32(1.0))
    assert np.allclose(vs, ret, rtol=1e-6, atol=1e-6) and np.allclose(pg, adv, rtol=1e-6, atol=1e-6)
    # and with lambda < 1 the trace coefficient is gamma * lambda: the GAE return
    vs, _ = orc.vtrace(zero, r, v, d, b, cfg.gamma, 0.9, 1.0, 1.0)
    adv, ret = orc.gae(r, v, d, b, np.float32(cfg.gamma), np.float32(0.9))
    assert np.allclose(vs, ret, rtol=1e-6, atol=1e-6)


def test_limits_of_the_truncation_levels():
    lr, r, v, d, b = _inputs(seed=5)
    g = 0.9 * (1.0 - (d != 0))
    vnext = np.vstack([v[1:], b[None]]).astype(np.float64)
    rho = np.minimum(1.0, np.exp(lr.astype(np.float64)))
    # c_bar = 0: no trace, vs_t = V_t + rho_t (one-step TD error)
    vs, pg = orc.vtrace(lr, r, v, d, b, 0.9, 1.0, 1.0, 0.0)
    assert np.allclose(vs, v + rho * (r + g * vnext - v), rtol=1e-6, atol=1e-6)
    # rho_bar = 0: nothing is learnt from the off-policy data: vs = V, pg = 0
    vs, pg = orc.vtrace(lr, r, v, d, b, 0.9, 1.0, 0.0, 1.0)
    assert np.array_equal(vs, v) and np.all(pg == 0)
    # truncation only binds above the level: ratios below both levels behave as untruncated
    small = np.minimum(lr, -0.01)
    a = orc.vtrace(small, r, v, d, b, 0.9, 1.0, 1.0, 1.0)
    bb = orc.vtrace(small, r, v, d, b, 0.9, 1.0, 50.0, 70.0)
    assert np.array_equal(a[0], bb[0]) and np.array_equal(a[1], bb[1])


def test_a_done_cuts_trace_and_bootstrap():
    lr, r, v, d, b = _inputs(T=12, N=5, seed=9, p_done=0.0)
    d[6] = 1
    vs1, pg1 = orc.vtrace(lr, r, v, d, b, 0.97, 1.0, 1.0, 1.0)
    lr2, r2, v2, b2 = lr.copy(), r.copy(), v.copy(), b + 3.0
    lr2[7:] += 0.4; r2[7:] -= 1.0; v2[7:] *= 2.0
    vs2, pg2 = orc.vtrace(lr2, r2, v2, d, b2, 0.97, 1.0, 1.0, 1.0)
    assert np.array_equal(vs1[:7], vs2[:7]) and np.array_equal(pg1[:7], pg2[:7])
    assert not np.array_equal(vs1[7:], vs2[7:])
    # T = 1 and all-done storages
    one = orc.vtrace(lr[:1], r[:1], v[:1], np.zeros_like(d[:1]), b, 0.97, 1.0, 1.0, 1.0)
    rho = np.minimum(1.0, np.exp(lr[0].astype(np.float64)))
    assert np.allclose(one[0][0], v[0] + rho * (r[0] + 0.97 * b - v[0]), rtol=1e-6, atol=1e-6)
    alld = orc.vtrace(lr, r, v, np.ones_like(d), b, 0.97, 1.0, 1.0, 1.0)
    rho_all = np.minimum(1.0, np.exp(lr.astype(np.float64)))
    assert np.allclose(alld[0], v + rho_all * (r - v), rtol=1e-6, atol=1e-6)
