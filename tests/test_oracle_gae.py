"""Pins for the oracle's advantage / return recurrence (Section 3, n-step return)."""
import os

import numpy as np

import hts_workloads as wl
from oracle import hts_oracle as orc

GOLD = os.path.join(os.path.dirname(__file__), "golden", "gae_worked_example.txt")


def _f32(*a):
    return [np.asarray(x, np.float32) for x in a]


def test_hand_worked_example():
    rows = [l.split() for l in open(GOLD) if l.strip() and not l.startswith("#")]
    r, v, b = _f32([[1], [0], [2]], [[0.5], [1], [0]], [4])
    for case, dones in (("nodone", [0, 0, 0]), ("done1", [0, 1, 0])):
        adv, ret = orc.gae(r, v, np.array(dones, np.uint8)[:, None], b, 0.5, 0.5)
        for name, t, a_exp, r_exp in rows:
            if name == case:
                assert adv[int(t), 0] == float(a_exp) and ret[int(t), 0] == float(r_exp)


def test_lambda_one_is_n_step_return():
    g = np.random.default_rng(0)
    T, N, gamma = 7, 5, 0.9
    r, v, b = _f32(g.standard_normal((T, N)), g.standard_normal((T, N)), g.standard_normal(N))
    adv, ret = orc.gae(r, v, np.zeros((T, N), np.uint8), b, gamma, 1.0)
    for t in range(T):
        n = T - t
        exp = sum(gamma**i * r[t + i].astype(np.float64) for i in range(n)) + gamma**n * b.astype(np.float64)
        np.testing.assert_allclose(ret[t], exp, rtol=1e-12, atol=1e-12)
        np.testing.assert_allclose(adv[t], exp - v[t], rtol=1e-12, atol=1e-12)


def test_general_lambda_is_discounted_sum_of_td_residuals():
    g = np.random.default_rng(1)
    T, N, gamma, lam = 9, 4, 0.97, 0.8
    r, v, b = _f32(g.standard_normal((T, N)), g.standard_normal((T, N)), g.standard_normal(N))
    adv, _ = orc.gae(r, v, np.zeros((T, N), np.uint8), b, gamma, lam)
    vnext = np.concatenate([v[1:], b[None]]).astype(np.float64)
    delta = r + gamma * vnext - v
    for t in range(T):
        exp = sum((gamma * lam) ** l * delta[t + l] for l in range(T - t))
        np.testing.assert_allclose(adv[t], exp, rtol=1e-12, atol=1e-12)


def test_lambda_zero_gamma_zero_all_done_and_T1():
    g = np.random.default_rng(2)
    T, N = 6, 3
    r, v, b = _f32(g.standard_normal((T, N)), g.standard_normal((T, N)), g.standard_normal(N))
    d = (g.random((T, N)) < 0.3).astype(np.uint8)
    vnext = np.concatenate([v[1:], b[None]]).astype(np.float64)
    adv, ret = orc.gae(r, v, d, b, 0.9, 0.0)
    np.testing.assert_allclose(adv, r + 0.9 * (1 - d) * vnext - v, rtol=1e-13, atol=1e-13)
    adv, ret = orc.gae(r, v, d, b, 0.0, 0.7)
    np.testing.assert_allclose(adv, r.astype(np.float64) - v, atol=1e-15)
    np.testing.assert_allclose(ret, r, atol=1e-15)
    adv1, _ = orc.gae(r, v, np.ones((T, N), np.uint8), b, 0.9, 0.7)
    np.testing.assert_allclose(adv1, adv, atol=1e-15)
    a, q = orc.gae(r[:1], v[:1], np.zeros((1, N), np.uint8), b, 0.5, 0.3)
    np.testing.assert_allclose(a[0], r[0] + 0.5 * b.astype(np.float64) - v[0], atol=1e-15)


def test_done_blocks_everything_after_it():
    g = np.random.default_rng(3)
    T, N, td = 8, 2, 4
    r, v, b = _f32(g.standard_normal((T, N)), g.standard_normal((T, N)), g.standard_normal(N))
    d = np.zeros((T, N), np.uint8); d[td, 0] = 1
    a0, r0 = orc.gae(r, v, d, b, 0.95, 0.9)
    r2, v2, b2 = r.copy(), v.copy(), b + 5
    r2[td + 1:] += 3; v2[td + 1:] -= 2
    a1, r1 = orc.gae(r2, v2, d, b2, 0.95, 0.9)
    assert np.array_equal(a0[:td + 1, 0], a1[:td + 1, 0]) and np.array_equal(r0[:td + 1, 0], r1[:td + 1, 0])
    assert not np.array_equal(a0[:td + 1, 1], a1[:td + 1, 1])          # the other env has no done


def test_linearity_and_segment_identity():
    g = np.random.default_rng(4)
    T, N, gamma, lam = 12, 3, 0.99, 0.95
    r, v, b = _f32(g.standard_normal((T, N)), g.standard_normal((T, N)), g.standard_normal(N))
    d = (g.random((T, N)) < 0.2).astype(np.uint8)
    a, _ = orc.gae(r, v, d, b, gamma, lam)
    a2, _ = orc.gae(2 * r, 2 * v, d, 2 * b, gamma, lam)
    np.testing.assert_allclose(a2, 2 * a, rtol=1e-12, atol=1e-12)
    # A_t = S_t + P_t * A_{t1}: S from a scan of rows [t0,t1) alone whose bootstrap is V_{t1}
    t0, t1 = 3, 8
    S, _ = orc.gae(r[t0:t1], v[t0:t1], d[t0:t1], v[t1], gamma, lam)
    for t in range(t0, t1):
        P = np.prod(gamma * lam * (1.0 - d[t:t1]), axis=0)
        np.testing.assert_allclose(a[t], S[t - t0] + P * a[t1], rtol=1e-12, atol=1e-12)


def test_config_shapes_run():
    cfg = wl.CONFIGS[2]
    r, v, d, b = wl.make_rollout(cfg)
    adv, ret = orc.gae(r, v, d, b, cfg.gamma, cfg.lam)
    assert adv.shape == (cfg.T, cfg.N) and np.isfinite(adv).all()
    np.testing.assert_allclose(ret, adv + v, rtol=1e-14, atol=1e-14)
