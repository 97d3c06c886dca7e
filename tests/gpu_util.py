"""Helpers of the GPU parity tests: run the CUDA library on seeded inputs."""
import numpy as np
import torch

import hts_workloads as wl
import paper_2012_09849_b200 as hts


def rel_err(got, ref):
    """max over elements of |got-ref| / max(|ref|, rms(ref)): relative error with the tensor's
    rms as the floor, so that values crossing zero do not blow the ratio up."""
    ref = np.asarray(ref, dtype=np.float64)
    got = np.asarray(got, dtype=np.float64)
    floor = float(np.sqrt(np.mean(ref ** 2))) if ref.size else 0.0
    den = np.maximum(np.abs(ref), max(floor, 1e-30))
    return float(np.max(np.abs(got - ref) / den)) if ref.size else 0.0


class Policy:
    """A context plus device copies of one config's weights."""

    def __init__(self, cfg, params=None, max_batch=None):
        self.cfg = cfg
        self.params = wl.make_weights(cfg) if params is None else params
        self.dtype = hts.HTS_DTYPE_FP32 if cfg.weight_dtype == "fp32" else hts.HTS_DTYPE_BF16
        self.max_batch = max_batch or cfg.N
        self.ctx = hts.hts_policy_create(cfg.C, cfg.H, cfg.W, cfg.A, self.dtype, self.max_batch)
        self.dev_w = hts.weights_to_device(self.params, self.dtype)
        hts.hts_policy_load_weights(self.ctx, self.dev_w)

    def step(self, obs, env_ids, t, seed, t_per_env=None, want_logits=True):
        n = obs.shape[0]
        d_obs = torch.from_numpy(np.ascontiguousarray(obs)).cuda()
        d_ids = torch.from_numpy(np.ascontiguousarray(env_ids, dtype=np.int32)).cuda()
        d_t = None if t_per_env is None else torch.from_numpy(np.ascontiguousarray(t_per_env, dtype=np.int32)).cuda()
        act = torch.empty(n, dtype=torch.int32, device="cuda")
        logp, val, ent = (torch.empty(n, dtype=torch.float32, device="cuda") for _ in range(3))
        logits = torch.empty(n, self.cfg.A, dtype=torch.float32, device="cuda") if want_logits else None
        hts.hts_policy_step(self.ctx, d_obs, d_ids, d_t, t, seed, n, act, logp, val, ent, logits)
        torch.cuda.synchronize()
        assert hts.hts_last_async_error(self.ctx) == 0
        out = {"actions": act.cpu().numpy(), "logp": logp.cpu().numpy(), "values": val.cpu().numpy(),
               "entropy": ent.cpu().numpy()}
        if want_logits:
            out["logits"] = logits.cpu().numpy()
        return out

    def activation(self, layer, n):
        g = self.cfg
        h1, w1 = wl.conv_out(g.H, 8, 4), wl.conv_out(g.W, 8, 4)
        h2, w2 = wl.conv_out(h1, 4, 2), wl.conv_out(w1, 4, 2)
        h3, w3 = wl.conv_out(h2, 3, 1), wl.conv_out(w2, 3, 1)
        shape = {1: (n, 32, h1, w1), 2: (n, 64, h2, w2), 3: (n, 64, h3, w3), 4: (n, 512)}[layer]
        out = torch.empty(shape, dtype=torch.float32, device="cuda")
        hts.hts_policy_read_activation(self.ctx, layer, n, out)
        torch.cuda.synchronize()
        return out.cpu().numpy()

    def close(self):
        if self.ctx:
            hts.hts_policy_destroy(self.ctx)
            self.ctx = None


def gpu_gae(r, v, d, b, gamma, lam):
    T, N = r.shape
    adv = torch.empty(T, N, dtype=torch.float32, device="cuda")
    ret = torch.empty_like(adv)
    hts.hts_gae(torch.from_numpy(r).cuda(), torch.from_numpy(v).cuda(), torch.from_numpy(d).cuda(),
                torch.from_numpy(b).cuda(), gamma, lam, T, N, adv, ret)
    torch.cuda.synchronize()
    return adv.cpu().numpy(), ret.cpu().numpy()
