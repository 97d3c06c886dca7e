"""hts_policy_step_indexed: frames gathered from a state buffer by slot, outputs scattered to the same
slot of a storage row (the executor-facing form of the actor step), against the oracle and against the
dense entry point."""
import dataclasses

import numpy as np
import pytest
import torch

import hts_workloads as wl
import paper_2012_09849_b200 as hts
from oracle import hts_oracle as orc
from gpu_util import Policy, rel_err

pytestmark = pytest.mark.gpu


def run_indexed(pol, state, slots, env_ids, t, seed, pool, sentinel=-7.0):
    n = len(slots)
    d_state = torch.from_numpy(state).cuda()
    d_slots = torch.from_numpy(np.ascontiguousarray(slots, dtype=np.int32)).cuda()
    d_ids = torch.from_numpy(np.ascontiguousarray(env_ids, dtype=np.int32)).cuda()
    act = torch.full((pool,), int(sentinel), dtype=torch.int32, device="cuda")
    logp, val, ent = (torch.full((pool,), sentinel, dtype=torch.float32, device="cuda") for _ in range(3))
    hts.hts_policy_step_indexed(pol.ctx, d_state, pool, d_slots, d_ids, None, t, seed, n, act, logp, val, ent)
    torch.cuda.synchronize()
    return {"actions": act.cpu().numpy(), "logp": logp.cpu().numpy(), "values": val.cpu().numpy(),
            "entropy": ent.cpu().numpy()}


@pytest.mark.parametrize("ci,pool,n", [(1, 40, 16), (2, 300, 137), (4, 64, 50)])
def test_indexed_step_matches_oracle_and_dense_step(ci, pool, n):
    cfg = wl.CONFIGS[ci]
    pol = Policy(cfg, max_batch=max(n, 8))
    try:
        g = np.random.default_rng(100 + ci)
        state = wl.make_obs(cfg, pool, batch_index=9)
        slots = g.permutation(pool)[:n].astype(np.int32)                # a random subset of the pool, in random order
        env_ids = (1000 + slots).astype(np.int32)                       # global ids differ from the local slots
        got = run_indexed(pol, state, slots, env_ids, 5, 777, pool)
        assert hts.hts_last_async_error(pol.ctx) == 0
        # untouched slots keep their previous contents
        rest = np.setdiff1d(np.arange(pool), slots)
        for k in got:
            assert np.all(got[k][rest] == -7)
        # bit for bit the dense step on the gathered frames
        dense = pol.step(state[slots], env_ids, 5, 777, want_logits=False)
        for k in dense:
            assert np.array_equal(got[k][slots], dense[k]), k
        # and the oracle on a sample of rows
        rows = np.arange(n) if n <= 48 else np.sort(g.choice(n, 48, replace=False))
        ref = orc.policy_step(orc.Weights(pol.params), state[slots[rows]], env_ids[rows], 5, 777)
        tol = 1e-4 if cfg.weight_dtype == "fp32" else 2e-2
        assert rel_err(got["values"][slots[rows]], ref["values"]) <= tol
        safe = ref["gap"] > 1e-3 + 4 * tol * max(1.0, float(np.sqrt(np.mean(ref["logits"] ** 2))))
        assert np.array_equal(got["actions"][slots[rows]][safe], ref["actions"][safe])
    finally:
        pol.close()


def test_indexed_step_serves_a_pool_in_executor_batches():
    """Random executor batches over a permutation of the pool fill one storage row exactly as one full batch does."""
    cfg = dataclasses.replace(wl.CONFIGS[5], N=700)
    pool = cfg.N
    pol = Policy(cfg, max_batch=pool)
    try:
        g = np.random.default_rng(5)
        state = wl.make_obs(cfg, pool, batch_index=3)
        ids = np.arange(pool, dtype=np.int32)
        full = pol.step(state, ids, 11, 2024, want_logits=False)
        d_state = torch.from_numpy(state).cuda()
        act = torch.empty(pool, dtype=torch.int32, device="cuda")
        logp, val, ent = (torch.empty(pool, dtype=torch.float32, device="cuda") for _ in range(3))
        perm = g.permutation(pool).astype(np.int32)
        pos = 0
        while pos < pool:
            size = int(g.integers(1, 200))
            sl = np.ascontiguousarray(perm[pos:pos + size])
            d_sl = torch.from_numpy(sl).cuda()
            hts.hts_policy_step_indexed(pol.ctx, d_state, pool, d_sl, d_sl, None, 11, 2024, len(sl), act, logp, val, ent)
            pos += size
        torch.cuda.synchronize()
        assert hts.hts_last_async_error(pol.ctx) == 0
        assert np.array_equal(act.cpu().numpy(), full["actions"])
        assert np.array_equal(logp.cpu().numpy(), full["logp"])
        assert np.array_equal(val.cpu().numpy(), full["values"])
        assert np.array_equal(ent.cpu().numpy(), full["entropy"])
    finally:
        pol.close()


def test_indexed_step_reports_a_slot_outside_the_pool():
    cfg = wl.CONFIGS[2]
    pool, n = 32, 8
    pol = Policy(cfg, max_batch=n)
    try:
        state = wl.make_obs(cfg, pool, batch_index=1)
        slots = np.array([3, 5, 40, 7, -1, 9, 11, 13], dtype=np.int32)          # 40 and -1 are outside [0, 32)
        got = run_indexed(pol, state, slots, np.arange(n), 0, 1, pool)
        assert hts.hts_last_async_error(pol.ctx) == 1                           # HTS_ERR_INVALID_ARG, then cleared
        assert hts.hts_last_async_error(pol.ctx) == 0
        good = slots[(slots >= 0) & (slots < pool)]
        assert np.all(got["values"][good] != -7)
        rest = np.setdiff1d(np.arange(pool), good)
        assert np.all(got["values"][rest] == -7)
        # host-side refusals
        L = hts.lib()
        assert L.hts_policy_step_indexed(pol.ctx, 8, 0, 16, 24, None, 0, 0, 4, 32, 40, 48, 56, None) == 1   # empty pool
        assert L.hts_policy_step_indexed(pol.ctx, 8, 4, None, 24, None, 0, 0, 4, 32, 40, 48, 56, None) == 1 # no slots
    finally:
        pol.close()
