"""Pins for the oracle's policy-value network (Appendix F.1 / F.2)."""
import math

import numpy as np
import pytest
import torch
import torch.nn.functional as F

import hts_workloads as wl
from oracle import hts_oracle as orc


def _torch_forward(p, obs):
    t = {k: torch.from_numpy(np.asarray(v, dtype=np.float64)) for k, v in p.items()}
    x = torch.from_numpy(obs.astype(np.float64)) / 255.0
    x = F.relu(F.conv2d(x, t["conv1_w"], t["conv1_b"], stride=4))
    x = F.relu(F.conv2d(x, t["conv2_w"], t["conv2_b"], stride=2))
    x = F.relu(F.conv2d(x, t["conv3_w"], t["conv3_b"], stride=1))
    h = F.relu(F.linear(x.flatten(1), t["fc_w"], t["fc_b"]))
    return F.linear(h, t["pi_w"], t["pi_b"]).numpy(), F.linear(h, t["v_w"], t["v_b"])[:, 0].numpy(), x.numpy(), h.numpy()


@pytest.mark.parametrize("ci", [1, 4])
def test_forward_matches_library_composition(ci):
    cfg = wl.CONFIGS[ci]
    p = wl.make_weights(cfg)
    obs = wl.make_obs(cfg, 3)
    out = orc.policy_forward(orc.Weights(p), obs, taps=True)
    logits, value, conv3, h = _torch_forward(p, obs)
    np.testing.assert_allclose(out["logits"], logits, rtol=1e-10, atol=1e-10)
    np.testing.assert_allclose(out["value"], value, rtol=1e-10, atol=1e-10)
    np.testing.assert_allclose(out["conv3"], conv3, rtol=1e-10, atol=1e-10)
    np.testing.assert_allclose(out["fc"], h, rtol=1e-10, atol=1e-10)
    F_ = wl.flat_features(cfg.H, cfg.W)
    assert out["conv3"].reshape(3, -1).shape[1] == F_ == p["fc_w"].shape[1]


def test_input_is_scaled_by_255():
    cfg = wl.CONFIGS[1]
    p = {k: np.zeros_like(v) for k, v in wl.make_weights(cfg).items()}
    p["conv1_w"][:] = 1.0 / (cfg.C * 64)          # each conv1 output = mean of its patch
    obs = np.full((1, cfg.C, cfg.H, cfg.W), 255, np.uint8)
    out = orc.policy_forward(orc.Weights(p), obs, taps=True)
    np.testing.assert_allclose(out["conv1"], 1.0, rtol=1e-12)
    obs[:] = 51                                    # 51/255 = 0.2
    out = orc.policy_forward(orc.Weights(p), obs, taps=True)
    np.testing.assert_allclose(out["conv1"], 0.2, rtol=1e-12)


def test_positive_homogeneity_without_biases():
    cfg = wl.CONFIGS[2]
    p = wl.make_weights(cfg)
    for k in p:
        if k.endswith("_b"):
            p[k] = np.zeros_like(p[k])
    obs = (wl.make_obs(cfg, 2) // 2).astype(np.uint8)      # <= 127 so 2x stays in range
    w = orc.Weights(p)
    a, b = orc.policy_forward(w, obs), orc.policy_forward(w, (obs * 2).astype(np.uint8))
    np.testing.assert_allclose(b["logits"], 2 * a["logits"], rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(b["value"], 2 * a["value"], rtol=1e-10, atol=1e-12)


def test_zero_heads_give_uniform_policy():
    cfg = wl.CONFIGS[2]
    p = wl.make_weights(cfg)
    p["pi_w"] = np.zeros_like(p["pi_w"]); p["pi_b"] = np.zeros_like(p["pi_b"])
    obs = wl.make_obs(cfg, 2)
    out = orc.policy_step(orc.Weights(p), obs, np.array([5, 9], np.int32), 3, seed=11)
    np.testing.assert_allclose(out["entropy"], math.log(cfg.A), rtol=1e-12)
    np.testing.assert_allclose(out["logp"], -math.log(cfg.A), rtol=1e-12)


def test_flatten_order_is_channel_major():
    # a single non-zero FC weight at flat index c*H3*W3 + h*W3 + w must pick conv3[c,h,w]
    cfg = wl.CONFIGS[1]
    p = wl.make_weights(cfg)
    obs = wl.make_obs(cfg, 1)
    w = orc.Weights(p)
    conv3 = orc.policy_forward(w, obs, taps=True)["conv3"][0]
    c, h, ww = np.unravel_index(np.argmax(conv3), conv3.shape)
    p2 = dict(p)
    p2["fc_w"] = np.zeros_like(p["fc_w"]); p2["fc_b"] = np.zeros_like(p["fc_b"])
    p2["fc_w"][7, (c * 7 + h) * 7 + ww] = 1.0
    fc = orc.policy_forward(orc.Weights(p2), obs, taps=True)["fc"][0]
    assert fc[7] == conv3[c, h, ww] > 0 and np.count_nonzero(fc) == 1
