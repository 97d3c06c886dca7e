"""CUDA actor step against the CPU oracle, through the C ABI."""
import numpy as np
import pytest
import torch

import hts_workloads as wl
import paper_2012_09849_b200 as hts
from oracle import hts_oracle as orc
from gpu_util import Policy, rel_err

pytestmark = pytest.mark.gpu
TOL = {"fp32": 1e-4, "bf16": 2e-2}      # relative, floor = rms of the reference tensor
GAP = 1e-3                               # oracle top-two score gap above which actions must agree
GATE_COUNTS = []                         # (config, rows, flips, flips with gap > 1e-3, rows in the band, max row error)


def check_against_oracle(cfg, got, ref, tol):
    e_log, e_val = rel_err(got["logits"], ref["logits"]), rel_err(got["values"], ref["values"])
    assert e_log <= tol, f"logits rel err {e_log}"
    assert e_val <= tol, f"values rel err {e_val}"
    # entropy and log-prob are smooth functions of the logits: same budget, absolute (nats)
    scale = max(1.0, float(np.sqrt(np.mean(ref["logits"] ** 2))))
    assert np.abs(got["entropy"] - ref["entropy"]).max() <= 4 * tol * scale
    # The acceptance rule, literally: identical actions wherever the oracle's top-two margin exceeds 1e-3
    # (measured logit errors are ~1e-3 of a unit, and no row of any configuration has been seen to flip).
    # Below the margin either of the oracle's two best actions is correct.
    row_err = np.abs(got["logits"] - ref["logits"]).max(axis=1)
    flipped = got["actions"] != ref["actions"]
    literal = int(np.sum(flipped & (ref["gap"] > GAP)))
    band = int(np.sum((ref["gap"] > GAP) & (ref["gap"] <= GAP + 2 * row_err)))
    GATE_COUNTS.append((cfg.name, len(flipped), int(flipped.sum()), literal, band, float(row_err.max())))
    print(f"action gate {cfg.name}: rows {len(flipped)}, flips {int(flipped.sum())}, flips with gap>1e-3 {literal}, "
          f"rows with 1e-3 < gap <= 1e-3 + 2 row_err {band}, max row logit err {row_err.max():.2e}")
    assert literal == 0, "an action differs although the oracle's margin exceeds 1e-3"
    assert np.array_equal(got["actions"][flipped], ref["runner_up"][flipped]), "a flip must go to the runner-up"
    # log-prob of the action the GPU chose, from the oracle's distribution
    for e in np.flatnonzero(flipped)[:50]:
        lp, _ = orc.log_softmax(ref["logits"][e])
        assert abs(got["logp"][e] - lp[got["actions"][e]]) <= 4 * tol * scale
    same = ~flipped
    assert np.abs(got["logp"][same] - ref["logp"][same]).max() <= 4 * tol * scale
    return e_log, e_val


def check_sampler_on_gpu_logits(cfg, got, env_ids, ts, seed):
    """The distribution and the sampling decision, given the logits the GPU itself produced:
    here both sides see identical inputs, so only fp32 rounding of the score separates them."""
    n = got["logits"].shape[0]
    for e in range(n):
        lg = got["logits"][e].astype(np.float64)
        lp, ent = orc.log_softmax(lg)
        s = orc.sample(lg, seed, int(env_ids[e]), int(ts[e]))
        if s["gap"] > 1e-4:
            assert got["actions"][e] == s["action"], (e, s["gap"])
        else:
            assert got["actions"][e] in (s["action"], s["runner_up"])
        assert abs(got["logp"][e] - lp[got["actions"][e]]) <= 2e-5 * max(1.0, abs(lp[got["actions"][e]]))
        assert abs(got["entropy"][e] - ent) <= 2e-5 * max(1.0, ent)


@pytest.mark.parametrize("ci,n,steps", [(1, 16, (0, 1, 2, 3, 4)), (2, 256, (0, 1, 2, 3, 4)), (3, 1024, (0, 1, 77, 127)),
                                        (4, 512, (0, 1, 300, 511))])
def test_configs_against_oracle(ci, n, steps):
    """Every row of the batch, at every time step of the short configurations and at the first two, the last
    and one seeded middle time step of the long ones."""
    cfg = wl.CONFIGS[ci]
    pol = Policy(cfg)
    try:
        wt = orc.Weights(pol.params)
        env_ids = np.arange(n, dtype=np.int32)
        for t in steps:
            obs = wl.make_obs(cfg, n, batch_index=t)
            got = pol.step(obs, env_ids, t, seed=0xC0FFEE + ci)
            ref = orc.policy_step(wt, obs, env_ids, t, 0xC0FFEE + ci)
            check_against_oracle(cfg, got, ref, TOL[cfg.weight_dtype])
            rows = np.arange(n) if n <= 256 else np.sort(np.random.default_rng(ci + t).choice(n, 256, replace=False))
            check_sampler_on_gpu_logits(cfg, {k: v[rows] for k, v in got.items()}, env_ids[rows], np.full(len(rows), t),
                                        0xC0FFEE + ci)
    finally:
        pol.close()


@pytest.mark.parametrize("ci", [1, 2, 4])
def test_layer_taps_against_oracle(ci):
    cfg = wl.CONFIGS[ci]
    n = 5
    pol = Policy(cfg, max_batch=8)
    try:
        obs = wl.make_obs(cfg, n, batch_index=77)
        pol.step(obs, np.arange(n), 0, 1)
        ref = orc.policy_forward(orc.Weights(pol.params), obs, taps=True)
        for layer, name in ((1, "conv1"), (2, "conv2"), (3, "conv3"), (4, "fc")):
            err = rel_err(pol.activation(layer, n), ref[name])
            assert err <= TOL[cfg.weight_dtype], (name, err)
    finally:
        pol.close()


@pytest.mark.parametrize("n", [1, 2, 3, 31, 127, 128, 129, 200])
def test_ragged_batch_sizes(n):
    cfg = wl.CONFIGS[2]
    pol = Policy(cfg, max_batch=256)
    try:
        obs = wl.make_obs(cfg, n, batch_index=n)
        ids = np.arange(1000, 1000 + n, dtype=np.int32)
        got = pol.step(obs, ids, 3, 99)
        rows = np.arange(n) if n <= 48 else np.sort(np.random.default_rng(n).choice(n, 48, replace=False))
        ref = orc.policy_step(orc.Weights(pol.params), obs[rows], ids[rows], 3, 99)
        check_against_oracle(cfg, {k: v[rows] for k, v in got.items()}, ref, TOL["bf16"])
    finally:
        pol.close()


@pytest.mark.parametrize("C,H,W,n", [(4, 64, 96, 77),     # 4 channels, width not 84: generic-width tensor-memory conv1; FC split 8
                                     (8, 84, 84, 33),     # 8 channels: shared-memory conv1 with two planes per tap
                                     (4, 36, 44, 150),    # image smaller than one 128-pixel tile: shared-memory conv1
                                     (4, 100, 84, 41),    # tiles straddle environments at other offsets (24 x 20 outputs)
                                     (4, 200, 252, 9)])   # widest frames: hidden grids of 25 x 31 and 23 x 30 positions
def test_other_frame_shapes(C, H, W, n):
    import dataclasses
    cfg = dataclasses.replace(wl.CONFIGS[2], C=C, H=H, W=W)
    pol = Policy(cfg, max_batch=n)
    try:
        obs = wl.make_obs(cfg, n, batch_index=H + W)
        ids = np.arange(500, 500 + n, dtype=np.int32)
        got = pol.step(obs, ids, 2, 4242)
        rows = np.arange(n) if n <= 40 else np.sort(np.random.default_rng(n).choice(n, 40, replace=False))
        wt = orc.Weights(pol.params)
        ref = orc.policy_step(wt, obs[rows], ids[rows], 2, 4242)
        check_against_oracle(cfg, {k: v[rows] for k, v in got.items()}, ref, TOL["bf16"])
        taps = orc.policy_forward(wt, obs[rows[:4]], taps=True)
        m = int(rows[3]) + 1
        for layer, name in ((1, "conv1"), (2, "conv2"), (3, "conv3")):
            err = rel_err(pol.activation(layer, m)[rows[:4]], taps[name])
            assert err <= TOL["bf16"], (name, err)
    finally:
        pol.close()


@pytest.mark.parametrize("A,dtype", [(1, "bf16"), (64, "bf16"), (1, "fp32"), (64, "fp32"), (33, "bf16")])
def test_extreme_action_counts(A, dtype):
    """One action (the sampler has no choice, entropy 0) and the largest head the library takes."""
    import dataclasses
    cfg = dataclasses.replace(wl.CONFIGS[2], A=A, weight_dtype=dtype)
    n = 21
    pol = Policy(cfg, max_batch=n)
    try:
        obs = wl.make_obs(cfg, n, batch_index=A)
        ids = np.arange(70, 70 + n, dtype=np.int32)
        got = pol.step(obs, ids, 4, 555)
        ref = orc.policy_step(orc.Weights(pol.params), obs, ids, 4, 555)
        check_against_oracle(cfg, got, ref, TOL[dtype])
        check_sampler_on_gpu_logits(cfg, got, ids, np.full(n, 4), 555)
        if A == 1:
            assert np.all(got["actions"] == 0) and np.all(got["logp"] == 0.0) and np.all(got["entropy"] == 0.0)
    finally:
        pol.close()


def test_uniform_stream_is_bit_exact():
    n, A, seed = 777, 19, 0xFEDCBA9876543210
    g = np.random.default_rng(0)
    ids = g.integers(0, 2**31 - 1, n).astype(np.int32)
    ts = g.integers(0, 100000, n).astype(np.int32)
    out = torch.empty(n, A, dtype=torch.float32, device="cuda")
    hts.hts_action_uniforms(torch.from_numpy(ids).cuda(), torch.from_numpy(ts).cuda(), 0, seed, n, A, out)
    torch.cuda.synchronize()
    got = out.cpu().numpy()
    for e in range(n):
        _, u = orc.action_uniforms(seed, int(ids[e]), int(ts[e]), A)
        assert np.array_equal(got[e].astype(np.float64), u)
    out2 = torch.empty(n, A, dtype=torch.float32, device="cuda")
    hts.hts_action_uniforms(torch.from_numpy(ids).cuda(), None, 5, seed, n, A, out2)
    torch.cuda.synchronize()
    _, u = orc.action_uniforms(seed, int(ids[3]), 5, A)
    assert np.array_equal(out2.cpu().numpy()[3].astype(np.float64), u)


def test_uniform_policy_actions_follow_the_uniforms_exactly():
    # zero policy head: every logit equal, so the action is the argmax of the uniforms alone
    cfg = wl.CONFIGS[2]
    p = wl.make_weights(cfg)
    p["pi_w"] = np.zeros_like(p["pi_w"]); p["pi_b"] = np.zeros_like(p["pi_b"])
    pol = Policy(cfg, params=p, max_batch=64)
    try:
        n = 64
        ids = np.arange(5000, 5000 + n, dtype=np.int32)
        got = pol.step(wl.make_obs(cfg, n), ids, 9, 4242)
        for e in range(n):
            _, u = orc.action_uniforms(4242, int(ids[e]), 9, cfg.A)
            assert got["actions"][e] == int(np.argmax(u))
        assert np.allclose(got["entropy"], np.log(cfg.A), rtol=1e-6)
        assert np.allclose(got["logp"], -np.log(cfg.A), rtol=1e-6)
    finally:
        pol.close()


def test_batch_grouping_does_not_change_any_output_bit():
    """Determinism invariant (Section 4.1; Table 4: identical scores for 1/4/8/16 actors): serving the
    pool in random executor batches over a random permutation gives the bits of one full batch."""
    cfg = wl.CONFIGS[5]
    pool = 8192
    pol = Policy(cfg, max_batch=pool)
    try:
        obs = wl.make_obs(cfg, pool)
        ids = np.arange(pool, dtype=np.int32)
        full = pol.step(obs, ids, 11, 2020)
        parts = {k: np.empty_like(v) for k, v in full.items()}
        sizes = []
        for batch in wl.make_async_batches(cfg, pool, 4096):
            out = pol.step(obs[batch], batch, 11, 2020)
            sizes.append(len(batch))
            for k in parts:
                parts[k][batch] = out[k]
        for batch in (ids[:1], ids[5:7], ids[100:103]):          # the smallest batches
            out = pol.step(obs[batch], batch, 11, 2020)
            for k in parts:
                assert np.array_equal(out[k].view(np.int32), full[k][batch].view(np.int32))
        assert len(sizes) >= 2
        for k in full:
            assert np.array_equal(parts[k].view(np.int32), full[k].view(np.int32)), k
        # and the full batch itself agrees with the oracle on a sample of rows
        rows = np.sort(np.random.default_rng(1).choice(pool, 96, replace=False))
        ref = orc.policy_step(orc.Weights(pol.params), obs[rows], ids[rows], 11, 2020)
        check_against_oracle(cfg, {k: v[rows] for k, v in full.items()}, ref, TOL["bf16"])
    finally:
        pol.close()


def test_per_env_time_index_and_duplicate_ids():
    cfg = wl.CONFIGS[2]
    pol = Policy(cfg, max_batch=16)
    try:
        n = 12
        obs = wl.make_obs(cfg, n)
        obs[7] = obs[2]
        ids = np.array([3, 8, 5, 1, 9, 4, 0, 5, 2, 6, 7, 10], np.int32)       # 5 appears twice
        ts = np.array([0, 1, 2, 3, 4, 5, 6, 2, 8, 9, 10, 11], np.int32)
        got = pol.step(obs, ids, 0, 77, t_per_env=ts)
        for k in got:                                              # same (obs, env_id, t) => same row
            assert np.array_equal(got[k][7], got[k][2])
        ref = orc.policy_step(orc.Weights(pol.params), obs, ids, 0, 77, t_per_env=ts)
        check_against_oracle(cfg, got, ref, TOL["bf16"])
        same_t = pol.step(obs, ids, 4, 77)
        assert same_t["actions"][4] == got["actions"][4]
    finally:
        pol.close()


def test_weights_can_be_reloaded():
    cfg = wl.CONFIGS[2]
    pol = Policy(cfg, max_batch=8)
    try:
        obs = wl.make_obs(cfg, 4)
        a = pol.step(obs, np.arange(4), 0, 1)
        p2 = wl.make_weights(cfg, sub=1)
        hts.hts_policy_load_weights(pol.ctx, hts.weights_to_device(p2, pol.dtype))
        b = pol.step(obs, np.arange(4), 0, 1)
        assert not np.array_equal(a["logits"], b["logits"])
        ref = orc.policy_step(orc.Weights(p2), obs, np.arange(4, dtype=np.int32), 0, 1)
        assert rel_err(b["logits"], ref["logits"]) <= TOL["bf16"]
    finally:
        pol.close()


def test_invalid_arguments_are_refused():
    cfg = wl.CONFIGS[2]
    ctx = hts.hts_policy_create(cfg.C, cfg.H, cfg.W, cfg.A, hts.HTS_DTYPE_BF16, 4)
    try:
        obs = torch.zeros(4, cfg.C, cfg.H, cfg.W, dtype=torch.uint8, device="cuda")
        ids = torch.zeros(4, dtype=torch.int32, device="cuda")
        act = torch.zeros(4, dtype=torch.int32, device="cuda")
        f = [torch.zeros(4, device="cuda") for _ in range(3)]
        with pytest.raises(hts.HtsError) as e:                    # weights not loaded yet
            hts.hts_policy_step(ctx, obs, ids, None, 0, 1, 4, act, *f)
        assert e.value.status == 6
        hts.hts_policy_load_weights(ctx, hts.weights_to_device(wl.make_weights(cfg), hts.HTS_DTYPE_BF16))
        for n in (0, 5):
            with pytest.raises(hts.HtsError) as e:
                hts.hts_policy_step(ctx, obs, ids, None, 0, 1, n, act, *f)
            assert e.value.status == 1
        with pytest.raises(hts.HtsError):
            hts.hts_policy_step(ctx, obs, ids, None, 0, 1, 4, act, f[0], f[0], f[2])
        with pytest.raises(hts.HtsError):
            hts.hts_policy_step(ctx, None, ids, None, 0, 1, 4, act, *f)
        # frames of a tensor-core context must start on a 16-byte boundary (they are staged by bulk copies):
        # a byte-offset view is refused on the host, nothing is launched
        big = torch.zeros(obs.numel() + 16, dtype=torch.uint8, device="cuda")
        before = hts.hts_launch_count()
        with pytest.raises(hts.HtsError) as e:
            hts.hts_policy_step(ctx, big.data_ptr() + 4, ids, None, 0, 1, 4, act, *f)
        assert e.value.status == 1
        with pytest.raises(hts.HtsError) as e:
            hts.hts_policy_evaluate(ctx, big.data_ptr() + 4, act, 4, *f)
        assert e.value.status == 1
        assert hts.hts_launch_count() == before
        hts.hts_policy_step(ctx, obs, ids, None, 0, 1, 4, act, *f)
        torch.cuda.synchronize()
    finally:
        hts.hts_policy_destroy(ctx)


def test_host_buffer_entry_point_matches_device_entry_point():
    cfg = wl.CONFIGS[2]
    pol = Policy(cfg, max_batch=64)
    try:
        n = 50
        obs = wl.make_obs(cfg, n); ids = np.arange(n, dtype=np.int32)
        dev = pol.step(obs, ids, 2, 5)
        act = np.empty(n, np.int32); lp, va, en = (np.empty(n, np.float32) for _ in range(3))
        lg = np.empty((n, cfg.A), np.float32)
        hts.hts_policy_step_host(pol.ctx, obs, ids, None, 2, 5, n, act, lp, va, en, lg)
        assert np.array_equal(act, dev["actions"]) and np.array_equal(lg, dev["logits"])
        assert np.array_equal(lp, dev["logp"]) and np.array_equal(va, dev["values"])
    finally:
        pol.close()


def test_zz_action_gate_summary():
    """Prints, per configuration seen by the tests above, how many actions differ from the oracle's and how
    many of those rows have an oracle margin above 1e-3 (collected by check_against_oracle)."""
    if not GATE_COUNTS:
        pytest.skip("no oracle comparison ran in this session")
    agg = {}
    for name, rows, flips, literal, band, err in GATE_COUNTS:
        a = agg.setdefault(name, [0, 0, 0, 0, 0.0])
        a[0] += rows; a[1] += flips; a[2] += literal; a[3] += band; a[4] = max(a[4], err)
    for name, (rows, flips, literal, band, err) in sorted(agg.items()):
        print(f"ACTION-GATE {name}: rows={rows} flips={flips} flips_with_gap_above_1e-3={literal} band_rows={band} "
              f"max_row_logit_err={err:.3e}")
