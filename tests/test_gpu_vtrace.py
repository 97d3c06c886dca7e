"""CUDA V-trace / truncated-importance-sampling scan against the CPU oracle, through the C ABI."""
import numpy as np
import pytest
import torch

import hts_workloads as wl
import paper_2012_09849_b200 as hts
from oracle import hts_oracle as orc
from gpu_util import gpu_gae, rel_err

pytestmark = pytest.mark.gpu
TOL = 1e-5          # relative, floor = rms of the reference tensor


def gpu_vtrace(lr, r, v, d, b, gamma, lam, rho_bar, c_bar):
    T, N = r.shape
    vs = torch.empty(T, N, dtype=torch.float32, device="cuda")
    pg = torch.empty_like(vs)
    hts.hts_vtrace(torch.from_numpy(lr).cuda(), torch.from_numpy(r).cuda(), torch.from_numpy(v).cuda(),
                   torch.from_numpy(d).cuda(), torch.from_numpy(b).cuda(), gamma, lam, rho_bar, c_bar, T, N, vs, pg)
    torch.cuda.synchronize()
    return vs.cpu().numpy(), pg.cpu().numpy()


def log_rhos(T, N, seed, scale=0.5):
    return (np.random.default_rng(seed).standard_normal((T, N)) * scale).astype(np.float32)


def _check(lr, r, v, d, b, gamma, lam, rho_bar=1.0, c_bar=1.0):
    vs, pg = gpu_vtrace(lr, r, v, d, b, gamma, lam, rho_bar, c_bar)
    f = lambda x: float(np.float32(x))
    vs_ref, pg_ref = orc.vtrace(lr, r, v, d, b, f(gamma), f(lam), f(rho_bar), f(c_bar))
    assert rel_err(vs, vs_ref) <= TOL, rel_err(vs, vs_ref)
    assert rel_err(pg, pg_ref) <= TOL, rel_err(pg, pg_ref)
    return vs, pg


@pytest.mark.parametrize("ci", [1, 2, 3, 4])
def test_configs_full_size(ci):
    cfg = wl.CONFIGS[ci]
    r, v, d, b = wl.make_rollout(cfg)
    _check(log_rhos(cfg.T, cfg.N, ci), r, v, d, b, cfg.gamma, cfg.lam)


@pytest.mark.parametrize("T,N", [(1, 1), (1, 33), (5, 16), (7, 31), (8, 32), (9, 65), (37, 203), (128, 1000),
                                 (257, 129), (513, 40), (1000, 7)])
def test_ragged_shapes_and_several_super_chunks(T, N):
    cfg = wl.CONFIGS[3]
    r, v, d, b = wl.make_rollout(cfg, T=T, N=N, sub=T * 1000 + N)
    d = (np.random.default_rng(T + N).random((T, N)) < 0.1).astype(np.uint8)
    _check(log_rhos(T, N, T + 7 * N), r, v, d, b, 0.99, 0.95, rho_bar=1.5, c_bar=0.8)


@pytest.mark.parametrize("T,N", [(128, 32768), (33, 131076), (64, 65537)])
def test_wide_problems(T, N):
    cfg = wl.CONFIGS[4]
    r, v, d, b = wl.make_rollout(cfg, T=T, N=N, sub=9)
    d = (np.random.default_rng(T).random((T, N)) < 0.05).astype(np.uint8)
    _check(log_rhos(T, N, N), r, v, d, b, 0.993, 1.0)


def test_on_policy_untruncated_equals_the_advantage_scan():
    cfg = wl.CONFIGS[3]
    r, v, d, b = wl.make_rollout(cfg)
    zero = np.zeros_like(r)
    vs, pg = gpu_vtrace(zero, r, v, d, b, cfg.gamma, cfg.lam, 1.0, 1.0)
    adv, ret = gpu_gae(r, v, d, b, cfg.gamma, cfg.lam)
    assert rel_err(vs, ret) <= TOL
    # pg uses the untruncated lambda = 1 continuation only when lambda = 1; compare that case
    vs1, pg1 = gpu_vtrace(zero, r, v, d, b, cfg.gamma, 1.0, 1.0, 1.0)
    adv1, ret1 = gpu_gae(r, v, d, b, cfg.gamma, 1.0)
    assert rel_err(vs1, ret1) <= TOL and rel_err(pg1, adv1) <= TOL


def test_done_mask_indexing_is_bit_exact():
    # dyadic inputs, ratios that are powers of two and gamma = 1/2: every intermediate is exact in fp32 for short
    # episodes, so a wrong done index shows as a bit difference
    g = np.random.default_rng(5)
    T, N = 16, 4100
    r = g.integers(-4, 5, (T, N)).astype(np.float32)
    v = (g.integers(-8, 9, (T, N)) / 4).astype(np.float32)
    b = (g.integers(-8, 9, N) / 4).astype(np.float32)
    d = (g.random((T, N)) < 0.3).astype(np.uint8)
    d[5::6] = 1                                          # episodes of at most six steps: 4 + 2*6 fraction bits fit fp32
    lr = np.zeros((T, N), np.float32)                    # ratio 1 exactly; truncation levels 1/2 bind everywhere
    vs, pg = gpu_vtrace(lr, r, v, d, b, 0.5, 1.0, 0.5, 0.5)
    vs_ref, pg_ref = orc.vtrace(lr, r, v, d, b, 0.5, 1.0, 0.5, 0.5)
    assert np.array_equal(vs.view(np.int32), vs_ref.view(np.int32))
    assert np.array_equal(pg.view(np.int32), pg_ref.view(np.int32))


def test_invalid_arguments_are_refused():
    x = torch.zeros(4, 4, device="cuda"); d = torch.zeros(4, 4, dtype=torch.uint8, device="cuda"); b = torch.zeros(4, device="cuda")
    o1, o2 = torch.zeros_like(x), torch.zeros_like(x)
    for args in ((x, x, x, d, b, 0.9, 1.0, -1.0, 1.0, 4, 4, o1, o2), (x, x, x, d, b, 0.9, 1.0, 1.0, float("nan"), 4, 4, o1, o2),
                 (x, x, x, d, b, 1.5, 1.0, 1.0, 1.0, 4, 4, o1, o2), (x, x, x, d, b, 0.9, 1.0, 1.0, 1.0, 4, 4, o1, o1),
                 (None, x, x, d, b, 0.9, 1.0, 1.0, 1.0, 4, 4, o1, o2)):
        with pytest.raises(hts.HtsError) as e:
            hts.hts_vtrace(*args)
        assert e.value.status == 1
