"""Pins for the oracle's policy distribution, Philox generator and Gumbel-max sampler."""
import math
import os

import numpy as np
import pytest
import scipy.special
import scipy.stats

import hts_workloads as wl
from oracle import hts_oracle as orc


# ---------------------------------------------------------------- distribution
def test_softmax_properties():
    g = np.random.default_rng(0)
    for A in (1, 2, 6, 18, 19):
        logits = g.standard_normal(A) * 3
        lp, ent = orc.log_softmax(logits)
        assert abs(np.exp(lp).sum() - 1) < 1e-12
        assert -1e-12 <= ent <= math.log(A) + 1e-12
        lp2, ent2 = orc.log_softmax(logits + 123.456)
        np.testing.assert_allclose(lp, lp2, atol=1e-12)
        np.testing.assert_allclose(lp, scipy.special.log_softmax(logits), atol=1e-12)
        np.testing.assert_allclose(ent, scipy.stats.entropy(np.exp(lp)), atol=1e-12)


def test_two_action_closed_form():
    lp, ent = orc.log_softmax(np.array([0.0, math.log(3.0)]))      # p = (1/4, 3/4)
    np.testing.assert_allclose(np.exp(lp), [0.25, 0.75], rtol=1e-14)
    np.testing.assert_allclose(ent, -(0.25 * math.log(0.25) + 0.75 * math.log(0.75)), rtol=1e-14)


def test_softmax_survives_large_logits():
    lp, ent = orc.log_softmax(np.array([1000.0, 1000.0, -1000.0]))
    np.testing.assert_allclose(np.exp(lp), [0.5, 0.5, 0.0], atol=1e-300)
    np.testing.assert_allclose(ent, math.log(2), rtol=1e-12)   # 1000+ln2 costs 3 digits


# ---------------------------------------------------------------------- Philox
def _philox_bigint(ctr, key):
    """Second statement of Philox4x32-10 with Python integers, written round by
    round from the published description (multiply, split, xor, Weyl key bump)."""
    M = (0xD2511F53, 0xCD9E8D57)
    Wk = (0x9E3779B9, 0xBB67AE85)
    c = list(ctr); k = list(key)
    for r in range(10):
        prod0, prod1 = M[0] * c[0], M[1] * c[2]
        c = [((prod1 >> 32) ^ c[1] ^ k[0]) & 0xFFFFFFFF, prod1 & 0xFFFFFFFF,
             ((prod0 >> 32) ^ c[3] ^ k[1]) & 0xFFFFFFFF, prod0 & 0xFFFFFFFF]
        k = [(k[0] + Wk[0]) & 0xFFFFFFFF, (k[1] + Wk[1]) & 0xFFFFFFFF]
    return tuple(c)


def test_philox_matches_bigint_restatement():
    g = np.random.default_rng(7)
    cases = [((0, 0, 0, 0), (0, 0)), ((0xFFFFFFFF,) * 4, (0xFFFFFFFF,) * 2)]
    cases += [(tuple(int(v) for v in g.integers(0, 2**32, 4)), tuple(int(v) for v in g.integers(0, 2**32, 2)))
              for _ in range(200)]
    for ctr, key in cases:
        assert orc.philox4x32_10(ctr, key) == _philox_bigint(ctr, key)


def test_philox_matches_independent_library_implementation():
    """Bit-exact agreement with Triton's philox (10 rounds, 4x32), run by its CPU
    interpreter: an implementation of the published generator that the oracle does
    not use."""
    os.environ["TRITON_INTERPRET"] = "1"
    torch = pytest.importorskip("torch")
    triton = pytest.importorskip("triton")
    import triton.language as tl

    @triton.jit
    def kern(out, ctr, key, n: tl.constexpr):
        i = tl.arange(0, n)
        c0 = tl.load(ctr + i * 4 + 0).to(tl.uint32)
        c1 = tl.load(ctr + i * 4 + 1).to(tl.uint32)
        c2 = tl.load(ctr + i * 4 + 2).to(tl.uint32)
        c3 = tl.load(ctr + i * 4 + 3).to(tl.uint32)
        k0 = tl.load(key + i * 2 + 0).to(tl.uint32)
        k1 = tl.load(key + i * 2 + 1).to(tl.uint32)
        r0, r1, r2, r3 = tl.philox_impl(c0, c1, c2, c3, k0, k1)
        tl.store(out + i * 4 + 0, r0.to(tl.int32, bitcast=True))
        tl.store(out + i * 4 + 1, r1.to(tl.int32, bitcast=True))
        tl.store(out + i * 4 + 2, r2.to(tl.int32, bitcast=True))
        tl.store(out + i * 4 + 3, r3.to(tl.int32, bitcast=True))

    n = 64
    g = np.random.default_rng(8)
    ctr = g.integers(0, 2**32, (n, 4), dtype=np.uint64).astype(np.uint32)
    key = g.integers(0, 2**32, (n, 2), dtype=np.uint64).astype(np.uint32)
    ctr[0] = 0; key[0] = 0
    ctr[1] = 0xFFFFFFFF; key[1] = 0xFFFFFFFF
    ctr[2] = (3, 17, 2, 0); key[2] = (0xDEADBEEF, 0x1234)          # an (env_id, t, block, 0) style counter
    out = torch.zeros(n * 4, dtype=torch.int32)
    try:
        kern[(1,)](out, torch.from_numpy(ctr.view(np.int32).reshape(-1)),
                   torch.from_numpy(key.view(np.int32).reshape(-1)), n=n)
    except Exception as e:                                      # interpreter not usable here
        pytest.skip(f"triton interpreter unavailable: {e}")
    got = out.numpy().view(np.uint32).reshape(n, 4)
    for i in range(n):
        assert orc.philox4x32_10(ctr[i], key[i]) == tuple(int(v) for v in got[i])


def test_philox_sensitivity_to_every_input_word():
    base = orc.philox4x32_10((3, 5, 1, 0), (11, 13))
    for pos in range(6):
        ctr, key = [3, 5, 1, 0], [11, 13]
        if pos < 4:
            ctr[pos] += 1
        else:
            key[pos - 4] += 1
        other = orc.philox4x32_10(ctr, key)
        assert all(a != b for a, b in zip(base, other))


def test_uniform23_is_exact_open_interval_and_fp32_representable():
    for w in (0, 0xFF, 0x100, 0xFFFFFFFF, 0x80000000, 0x12345678):
        u = orc.uniform23(w)
        assert u == ((w >> 9) + 0.5) / 2**23
        assert 0.0 < u < 1.0
        assert float(np.float32(u)) == u
    assert orc.uniform23(0) == 2.0**-24 and orc.uniform23(0xFFFFFFFF) == 1 - 2.0**-24


def test_action_uniforms_use_block_and_lane():
    seed, env, t, A = 0x0123456789ABCDEF, 77, 12, 19
    words, u = orc.action_uniforms(seed, env, t, A)
    for a in range(A):
        blk = orc.philox4x32_10((env, t, a // 4, 0), (seed & 0xFFFFFFFF, seed >> 32))
        assert int(words[a]) == blk[a % 4]
        assert u[a] == orc.uniform23(blk[a % 4])


def test_uniform_statistics():
    us = np.concatenate([orc.action_uniforms(99, e, 0, 4096)[1] for e in range(256)])   # 2^20 uniforms
    assert abs(us.mean() - 0.5) < 1e-3
    counts = np.bincount((us * 256).astype(int), minlength=256)
    chi2 = ((counts - us.size / 256) ** 2 / (us.size / 256)).sum()
    assert chi2 < scipy.stats.chi2.ppf(1 - 1e-6, 255)


# --------------------------------------------------------------------- sampler
def test_gumbel_max_frequencies_follow_softmax():
    logits = np.array([0.3, -1.2, 2.0, 0.0, 1.1, -0.4])
    p = np.exp(orc.log_softmax(logits)[0])
    n = 60000
    counts = np.zeros(len(logits))
    for i in range(n):
        counts[orc.sample(logits, seed=2024, env_id=i % 300, t=i // 300)["action"]] += 1
    chi2 = ((counts - n * p) ** 2 / (n * p)).sum()
    assert chi2 < scipy.stats.chi2.ppf(1 - 1e-6, len(logits) - 1)


def test_sampler_scores_gap_and_dominant_logit():
    logits = np.array([0.0, 50.0, 0.0])
    s = orc.sample(logits, seed=1, env_id=2, t=3)
    assert s["action"] == 1                          # Gumbel noise never reaches +50 here
    _, u = orc.action_uniforms(1, 2, 3, 3)
    np.testing.assert_allclose(s["scores"], logits - np.log(-np.log(u)), rtol=1e-13)
    srt = np.sort(s["scores"])
    np.testing.assert_allclose(s["gap"], srt[-1] - srt[-2], rtol=1e-13)
    assert s["runner_up"] == int(np.argsort(s["scores"])[-2])
    assert orc.sample(np.array([0.7]), 1, 2, 3)["action"] == 0


def test_sampler_depends_only_on_seed_env_t():
    logits = np.linspace(-1, 1, 18)
    a = orc.sample(logits, 5, 10, 20)["action"]
    assert a == orc.sample(logits, 5, 10, 20)["action"]
    others = {orc.sample(logits, s, e, t)["action"] for s, e, t in
              [(6, 10, 20), (5, 11, 20), (5, 10, 21)] + [(5, 10, 100 + k) for k in range(40)]}
    assert len(others) > 1


def test_actions_invariant_under_batch_permutation_and_split():
    cfg = wl.CONFIGS[1]
    wt = orc.Weights(wl.make_weights(cfg))
    obs = wl.make_obs(cfg, 6)
    ids = np.array([4, 9, 2, 7, 7, 0], np.int32)              # a duplicate id is legal
    full = orc.policy_step(wt, obs, ids, 3, seed=42)
    perm = np.array([5, 3, 0, 4, 2, 1])
    pp = orc.policy_step(wt, obs[perm], ids[perm], 3, seed=42)
    for k in ("actions", "logp", "values", "entropy"):
        assert np.array_equal(pp[k], full[k][perm])
    a = orc.policy_step(wt, obs[:2], ids[:2], 3, seed=42)
    b = orc.policy_step(wt, obs[2:], ids[2:], 3, seed=42)
    assert np.array_equal(np.concatenate([a["actions"], b["actions"]]), full["actions"])
    tp = orc.policy_step(wt, obs, ids, 0, seed=42, t_per_env=np.full(6, 3, np.int32))
    assert np.array_equal(tp["actions"], full["actions"])
