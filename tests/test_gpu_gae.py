"""CUDA advantage scan against the CPU oracle, through the C ABI."""
import numpy as np
import pytest
import torch

import hts_workloads as wl
import paper_2012_09849_b200 as hts
from oracle import hts_oracle as orc
from gpu_util import gpu_gae, rel_err

pytestmark = pytest.mark.gpu
TOL = 1e-5          # relative, floor = rms of the reference tensor


def _check(r, v, d, b, gamma, lam):
    adv, ret = gpu_gae(r, v, d, b, gamma, lam)
    a_ref, r_ref = orc.gae(r, v, d, b, float(np.float32(gamma)), float(np.float32(lam)))
    assert rel_err(adv, a_ref) <= TOL, rel_err(adv, a_ref)
    assert rel_err(ret, r_ref) <= TOL, rel_err(ret, r_ref)
    return adv, ret


@pytest.mark.parametrize("ci", [1, 2, 3, 4])
def test_configs_full_size(ci):
    cfg = wl.CONFIGS[ci]
    _check(*wl.make_rollout(cfg), cfg.gamma, cfg.lam)


@pytest.mark.parametrize("T,N", [(1, 1), (1, 33), (5, 16), (7, 31), (8, 32), (9, 65), (37, 203), (128, 1000),
                                 (257, 129), (300, 70), (513, 40), (1000, 7)])
def test_ragged_shapes_and_several_super_chunks(T, N):
    cfg = wl.CONFIGS[3]
    r, v, d, b = wl.make_rollout(cfg, T=T, N=N, sub=T * 1000 + N)
    d = (np.random.default_rng(T + N).random((T, N)) < 0.1).astype(np.uint8)
    _check(r, v, d, b, 0.99, 0.95)


@pytest.mark.parametrize("T,N", [(128, 32768), (512, 8192), (33, 131076), (70, 65540)])
def test_wide_problems_take_the_vector_path(T, N):
    cfg = wl.CONFIGS[4]
    r, v, d, b = wl.make_rollout(cfg, T=T, N=N, sub=9)
    d = (np.random.default_rng(T).random((T, N)) < 0.05).astype(np.uint8)
    _check(r, v, d, b, 0.993, 0.95)


@pytest.mark.parametrize("T,N", [(512, 512), (128, 1024), (300, 70), (37, 203), (1100, 24)])
def test_narrow_blocks_give_the_bits_of_wide_ones(T, N):
    # few columns take 8-column blocks; the same columns inside a wide scalar problem take 32-column blocks.
    # Chunk boundaries are the same, so every output bit must be.
    cfg = wl.CONFIGS[4]
    r, v, d, b = wl.make_rollout(cfg, T=T, N=N, sub=77)
    d = (np.random.default_rng(T * 7 + N).random((T, N)) < 0.02).astype(np.uint8)
    adv, ret = _check(r, v, d, b, 0.993, 0.95)
    reps = -(-4801 // N)                                 # wide enough for 32-column blocks, odd width: scalar columns
    wide = [np.ascontiguousarray(np.tile(x, (1, reps))[:, :reps * N - 1]) for x in (r, v, d)]
    bw = np.ascontiguousarray(np.tile(b, reps)[:reps * N - 1])
    adv_w, ret_w = gpu_gae(wide[0], wide[1], wide[2], bw, 0.993, 0.95)
    assert np.array_equal(adv_w[:, :N].view(np.int32), adv.view(np.int32))
    assert np.array_equal(ret_w[:, :N].view(np.int32), ret.view(np.int32))


def test_unaligned_wide_problem_falls_back():
    cfg = wl.CONFIGS[3]
    T, N = 64, 65537                                     # N % 4 != 0: scalar columns
    r, v, d, b = wl.make_rollout(cfg, T=T, N=N, sub=3)
    _check(r, v, d, b, 0.99, 0.95)


def test_done_mask_indexing_is_bit_exact():
    # dyadic inputs and gamma = lambda = 1/2 make every intermediate exact in fp32 for short
    # episodes, so any wrong done index shows as a bit difference
    g = np.random.default_rng(5)
    T, N = 24, 4100
    r = g.integers(-4, 5, (T, N)).astype(np.float32)
    v = (g.integers(-8, 9, (T, N)) / 4).astype(np.float32)
    b = (g.integers(-8, 9, N) / 4).astype(np.float32)
    d = (g.random((T, N)) < 0.3).astype(np.uint8)
    d[::6] = 1                                           # episodes of at most 6 steps: <= 20 fraction bits
    adv, ret = gpu_gae(r, v, d, b, 0.5, 0.5)
    a_ref, r_ref = orc.gae(r, v, d, b, 0.5, 0.5)
    assert np.array_equal(adv.astype(np.float64), a_ref)
    assert np.array_equal(ret.astype(np.float64), r_ref)


def test_degenerate_parameters():
    cfg = wl.CONFIGS[2]
    r, v, d, b = wl.make_rollout(cfg, T=40, N=100)
    _check(r, v, d, b, 0.0, 0.7)
    _check(r, v, d, b, 0.9, 0.0)
    _check(r, v, d, b, 1.0, 1.0)
    _check(r, v, np.ones_like(d), b, 0.99, 0.95)
    _check(r, v, np.zeros_like(d), b, 0.99, 1.0)


def test_invalid_arguments_are_refused():
    x = torch.zeros(4, 4, device="cuda"); dd = torch.zeros(4, 4, dtype=torch.uint8, device="cuda")
    bb = torch.zeros(4, device="cuda"); o1 = torch.zeros(4, 4, device="cuda"); o2 = torch.zeros(4, 4, device="cuda")
    for bad in (dict(gamma=1.5), dict(lam=-0.1), dict(gamma=float("nan")), dict(T=0)):
        kw = dict(gamma=0.9, lam=0.9, T=4); kw.update(bad)
        with pytest.raises(hts.HtsError) as e:
            hts.hts_gae(x, x.clone(), dd, bb, kw["gamma"], kw["lam"], kw["T"], 4, o1, o2)
        assert e.value.status == 1
    with pytest.raises(hts.HtsError):                    # output aliases an input
        hts.hts_gae(x, x.clone(), dd, bb, 0.9, 0.9, 4, 4, x, o2)
    with pytest.raises(hts.HtsError):                    # outputs alias each other
        hts.hts_gae(x, x.clone(), dd, bb, 0.9, 0.9, 4, 4, o1, o1)


def test_host_buffer_entry_point():
    cfg = wl.CONFIGS[3]
    r, v, d, b = wl.make_rollout(cfg, T=50, N=333)
    adv = np.empty_like(r); ret = np.empty_like(r)
    hts.hts_gae_host(r, v, d, b, cfg.gamma, cfg.lam, 50, 333, adv, ret)
    a_ref, r_ref = orc.gae(r, v, d, b, float(np.float32(cfg.gamma)), float(np.float32(cfg.lam)))
    assert rel_err(adv, a_ref) <= TOL and rel_err(ret, r_ref) <= TOL
