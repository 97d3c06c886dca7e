"""Seeded synthetic inputs for the HTS-RL actor step and advantage scan.

This module only draws inputs.  It holds none of the method's arithmetic and is the
one piece shared by the CPU oracle's tests and the CUDA library's tests: both read
the very same arrays.  The shapes and value laws stand in for ALE Atari frames and
GFootball "extracted map" observations, which cannot be produced here.

Streams: every array comes from ``numpy.random.Generator(PCG64(SeedSequence(
[BASE_SEED, config_index, purpose, sub_index])))`` so that arrays are independent
of the order in which they are requested.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

BASE_SEED = 0x2012_0984_9000

# purposes (sub-streams)
_WEIGHTS, _OBS, _REWARDS, _DONES, _VALUES, _BOOT, _PERM, _SIZES = range(8)


@dataclass(frozen=True)
class Config:
    index: int
    name: str
    N: int                # environments
    T: int                # unroll length (rows of the rollout storage)
    C: int
    H: int
    W: int
    A: int                # number of actions
    weight_dtype: str     # "fp32" or "bf16"
    obs_law: str          # "uniform" (iid 0..255) or "sparse" (255 w.p. 0.02 else 0)
    p_reward: float
    p_done: float
    gamma: float
    lam: float


CONFIGS = {
    1: Config(1, "a2c_atari_tiny", 16, 5, 4, 84, 84, 6, "fp32", "uniform", 0.05, 0.02, 0.99, 1.0),
    2: Config(2, "a2c_atari", 256, 5, 4, 84, 84, 18, "bf16", "uniform", 0.05, 0.01, 0.99, 1.0),
    3: Config(3, "ppo_atari_large", 1024, 128, 4, 84, 84, 18, "bf16", "uniform", 0.03, 0.005, 0.99, 0.95),
    4: Config(4, "ppo_football", 512, 512, 16, 72, 96, 19, "bf16", "sparse", 0.001, 0.002, 0.993, 0.95),
    5: Config(5, "async_batching_sweep", 8192, 1, 4, 84, 84, 18, "bf16", "uniform", 0.0, 0.0, 0.99, 0.95),
}


def _rng(cfg_index: int, purpose: int, sub: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(
        np.random.SeedSequence([BASE_SEED, int(cfg_index), int(purpose), int(sub)])))


def conv_out(extent: int, k: int, s: int) -> int:
    return (extent - k) // s + 1


def flat_features(H: int, W: int) -> int:
    h, w = conv_out(H, 8, 4), conv_out(W, 8, 4)
    h, w = conv_out(h, 4, 2), conv_out(w, 4, 2)
    h, w = conv_out(h, 3, 1), conv_out(w, 3, 1)
    return 64 * h * w


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round fp32 to the nearest bf16 (ties to even); result kept as fp32 values."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).reshape(np.shape(x))


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """The 16-bit patterns of values that are already bf16-representable."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    assert not np.any(u & 0xFFFF), "value is not bf16-representable"
    return (u >> 16).astype(np.uint16).reshape(np.shape(x))


def make_weights(cfg: Config, sub: int = 0) -> dict:
    """He-normal weights N(0, 2/fan_in), biases U(-0.1, 0.1); fp32 arrays.  For a
    bf16 config every value is already rounded to bf16, so both sides see the
    exact same numbers."""
    g = _rng(cfg.index, _WEIGHTS, sub)
    F = flat_features(cfg.H, cfg.W)
    shapes = {
        "conv1_w": (32, cfg.C, 8, 8), "conv1_b": (32,),
        "conv2_w": (64, 32, 4, 4), "conv2_b": (64,),
        "conv3_w": (64, 64, 3, 3), "conv3_b": (64,),
        "fc_w": (512, F), "fc_b": (512,),
        "pi_w": (cfg.A, 512), "pi_b": (cfg.A,),
        "v_w": (1, 512), "v_b": (1,),
    }
    out = {}
    for name, shp in shapes.items():
        if name.endswith("_w"):
            fan_in = int(np.prod(shp[1:]))
            a = g.standard_normal(shp, dtype=np.float32) * np.float32(np.sqrt(2.0 / fan_in))
        else:
            a = g.uniform(-0.1, 0.1, size=shp).astype(np.float32)
        if cfg.weight_dtype == "bf16":
            a = round_to_bf16(a)
        out[name] = np.ascontiguousarray(a, dtype=np.float32)
    return out


def make_obs(cfg: Config, n: int, batch_index: int = 0) -> np.ndarray:
    """uint8 [n,C,H,W] observations for one actor step."""
    g = _rng(cfg.index, _OBS, batch_index)
    shp = (n, cfg.C, cfg.H, cfg.W)
    if cfg.obs_law == "uniform":
        return g.integers(0, 256, size=shp, dtype=np.uint8)
    if cfg.obs_law == "sparse":
        return np.where(g.random(shp, dtype=np.float32) < 0.02, 255, 0).astype(np.uint8)
    raise ValueError(cfg.obs_law)


def make_rollout(cfg: Config, T: int | None = None, N: int | None = None, sub: int = 0):
    """Stand-alone advantage-scan inputs: rewards in {-1,0,1}, Bernoulli dones,
    values and bootstrap iid N(0,1); time-major [T,N]."""
    T = cfg.T if T is None else T
    N = cfg.N if N is None else N
    gr, gd = _rng(cfg.index, _REWARDS, sub), _rng(cfg.index, _DONES, sub)
    gv, gb = _rng(cfg.index, _VALUES, sub), _rng(cfg.index, _BOOT, sub)
    nz = gr.random((T, N), dtype=np.float32) < cfg.p_reward
    sign = np.where(gr.random((T, N), dtype=np.float32) < 0.5, -1.0, 1.0)
    rewards = np.where(nz, sign, 0.0).astype(np.float32)
    dones = (gd.random((T, N), dtype=np.float32) < cfg.p_done).astype(np.uint8)
    values = gv.standard_normal((T, N), dtype=np.float32)
    bootstrap = gb.standard_normal((N,), dtype=np.float32)
    return rewards, values, dones, bootstrap


def make_async_batches(cfg: Config, pool: int, max_batch: int, sub: int = 0):
    """A random permutation of env ids 0..pool-1 cut into batches of random size
    1..max_batch: how asynchronous executors might hand observations to actors."""
    gp, gs = _rng(cfg.index, _PERM, sub), _rng(cfg.index, _SIZES, sub)
    perm = gp.permutation(pool).astype(np.int32)
    batches, i = [], 0
    while i < pool:
        sz = int(gs.integers(1, max_batch + 1))
        batches.append(perm[i:i + sz].copy())
        i += sz
    return batches
