"""ctypes front end of the plain-C oracle (``hts_oracle.c``).

TEST INFRASTRUCTURE ONLY.  The oracle states, in slow fp64 loops, what the actor
step and the advantage scan of HTS-RL (arXiv 2012.09849) compute.  It shares
nothing with the CUDA library; only tests, the smoke check and the CPU-baseline
leg of the benchmark call it.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "hts_oracle.c")
_LIB = os.path.join(_HERE, "libhts_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (OpenMP over environments)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"])
    return _LIB


class _Weights(C.Structure):
    _fields_ = [(name, C.c_void_p) for name in (
        "conv1_w", "conv1_b", "conv2_w", "conv2_b", "conv3_w", "conv3_b",
        "fc_w", "fc_b", "pi_w", "pi_b", "v_w", "v_b")]


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.hts_oracle_uniform23.restype = C.c_double
        _lib.hts_oracle_uniform23.argtypes = [C.c_uint32]
        _lib.hts_oracle_sample.restype = C.c_int32
        _lib.hts_oracle_conv_out.restype = C.c_int
        _lib.hts_oracle_flat_features.restype = C.c_int
        _lib.hts_oracle_num_threads.restype = C.c_int
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _f64(a):
    return np.ascontiguousarray(np.asarray(a, dtype=np.float64))


def num_threads() -> int:
    return int(lib().hts_oracle_num_threads())


def conv_out(extent: int, k: int, s: int) -> int:
    return int(lib().hts_oracle_conv_out(extent, k, s))


def conv2d(x, w, b, stride: int, relu: bool):
    """x [C,H,W], w [O,C,k,k], b [O] -> y [O,Ho,Wo]; cross-correlation, no padding."""
    x, w, b = _f64(x), _f64(w), _f64(b)
    Cc, H, W = x.shape
    O, C2, k, k2 = w.shape
    assert C2 == Cc and k == k2 and b.shape == (O,)
    Ho, Wo = conv_out(H, k, stride), conv_out(W, k, stride)
    y = np.empty((O, Ho, Wo), dtype=np.float64)
    lib().hts_oracle_conv2d(_p(x), Cc, H, W, _p(w), _p(b), O, k, stride, int(relu), _p(y))
    return y


def linear(x, w, b, relu: bool):
    x, w, b = _f64(x), _f64(w), _f64(b)
    O, I = w.shape
    y = np.empty(O, dtype=np.float64)
    lib().hts_oracle_linear(_p(x), I, _p(w), _p(b), O, int(relu), _p(y))
    return y


class Weights:
    """fp64 copies of the twelve parameter tensors (PyTorch OIHW / [out,in] layout)."""
    NAMES = ("conv1_w", "conv1_b", "conv2_w", "conv2_b", "conv3_w", "conv3_b",
             "fc_w", "fc_b", "pi_w", "pi_b", "v_w", "v_b")

    def __init__(self, params: dict):
        self.arr = {k: _f64(params[k]) for k in self.NAMES}
        self.A = self.arr["pi_w"].shape[0]
        self.C = self.arr["conv1_w"].shape[1]
        self.c = _Weights(**{k: _p(v) for k, v in self.arr.items()})


def policy_forward(wt: Weights, obs: np.ndarray, taps: bool = False):
    """obs u8 [n,C,H,W] -> dict(logits [n,A], value [n], optional layer taps)."""
    obs = np.ascontiguousarray(obs, dtype=np.uint8)
    n, Cc, H, W = obs.shape
    assert Cc == wt.C
    A = wt.A
    h1, w1 = conv_out(H, 8, 4), conv_out(W, 8, 4)
    h2, w2 = conv_out(h1, 4, 2), conv_out(w1, 4, 2)
    h3, w3 = conv_out(h2, 3, 1), conv_out(w2, 3, 1)
    assert wt.arr["fc_w"].shape == (512, 64 * h3 * w3)
    out = {"logits": np.empty((n, A)), "value": np.empty(n)}
    t1 = t2 = t3 = t4 = None
    if taps:
        t1 = np.empty((n, 32, h1, w1)); t2 = np.empty((n, 64, h2, w2))
        t3 = np.empty((n, 64, h3, w3)); t4 = np.empty((n, 512))
        out.update(conv1=t1, conv2=t2, conv3=t3, fc=t4)
    lib().hts_oracle_policy_forward(C.byref(wt.c), _p(obs), n, Cc, H, W, A,
                                    _p(out["logits"]), _p(out["value"]),
                                    _p(t1), _p(t2), _p(t3), _p(t4))
    return out


def log_softmax(logits):
    """logits [A] -> (log pi [A], entropy) in nats (Eq. 3's H)."""
    logits = _f64(logits)
    A = logits.shape[0]
    lp = np.empty(A)
    ent = C.c_double()
    lib().hts_oracle_log_softmax(_p(logits), A, _p(lp), C.byref(ent))
    return lp, ent.value


def philox4x32_10(ctr, key):
    c = (C.c_uint32 * 4)(*[int(v) & 0xFFFFFFFF for v in ctr])
    k = (C.c_uint32 * 2)(*[int(v) & 0xFFFFFFFF for v in key])
    o = (C.c_uint32 * 4)()
    lib().hts_oracle_philox4x32_10(c, k, o)
    return tuple(int(v) for v in o)


def uniform23(word: int) -> float:
    return float(lib().hts_oracle_uniform23(C.c_uint32(int(word) & 0xFFFFFFFF)))


def action_uniforms(seed: int, env_id: int, t: int, A: int):
    """-> (words u32 [A], uniforms f64 [A]) for (seed, env_id, t)."""
    words = np.empty(A, dtype=np.uint32)
    u = np.empty(A, dtype=np.float64)
    lib().hts_oracle_action_uniforms(C.c_uint64(seed), C.c_int32(env_id), C.c_int32(t), A,
                                     _p(words), _p(u))
    return words, u


def sample(logits, seed: int, env_id: int, t: int):
    """-> dict(action, scores [A], gap, runner_up): Gumbel-max on (seed, env_id, t)."""
    logits = _f64(logits)
    A = logits.shape[0]
    scores = np.empty(A)
    gap = C.c_double()
    ru = C.c_int32()
    a = lib().hts_oracle_sample(_p(logits), A, C.c_uint64(seed), C.c_int32(env_id),
                                C.c_int32(t), _p(scores), C.byref(gap), C.byref(ru))
    return {"action": int(a), "scores": scores, "gap": gap.value, "runner_up": ru.value}


def policy_step(wt: Weights, obs, env_ids, t, seed: int, t_per_env=None):
    """The whole actor step on a batch. Returns a dict of per-env arrays."""
    obs = np.ascontiguousarray(obs, dtype=np.uint8)
    n, Cc, H, W = obs.shape
    env_ids = np.ascontiguousarray(env_ids, dtype=np.int32)
    assert env_ids.shape == (n,)
    tp = None if t_per_env is None else np.ascontiguousarray(t_per_env, dtype=np.int32)
    A = wt.A
    out = {"actions": np.empty(n, np.int32), "logp": np.empty(n), "values": np.empty(n),
           "entropy": np.empty(n), "logits": np.empty((n, A)), "gap": np.empty(n),
           "runner_up": np.empty(n, np.int32)}
    lib().hts_oracle_policy_step(C.byref(wt.c), _p(obs), _p(env_ids), _p(tp), C.c_int32(int(t)),
                                 C.c_uint64(seed), n, Cc, H, W, A,
                                 _p(out["actions"]), _p(out["logp"]), _p(out["values"]),
                                 _p(out["entropy"]), _p(out["logits"]), _p(out["gap"]),
                                 _p(out["runner_up"]))
    return out


def gae(rewards, values, dones, bootstrap, gamma: float, lam: float):
    """[T,N] fp32 rewards/values, u8 dones, [N] bootstrap -> (adv, ret) fp64 [T,N]."""
    r = np.ascontiguousarray(rewards, dtype=np.float32)
    v = np.ascontiguousarray(values, dtype=np.float32)
    d = np.ascontiguousarray(dones, dtype=np.uint8)
    b = np.ascontiguousarray(bootstrap, dtype=np.float32)
    T, N = r.shape
    assert v.shape == (T, N) and d.shape == (T, N) and b.shape == (N,)
    adv = np.empty((T, N)); ret = np.empty((T, N))
    lib().hts_oracle_gae(_p(r), _p(v), _p(d), _p(b), C.c_double(gamma), C.c_double(lam),
                         T, N, _p(adv), _p(ret))
    return adv, ret


def evaluate_actions(wt: Weights, obs, actions):
    """What the learner re-evaluates on stored transitions (Section 3, Eq. 3/4): for each row the
    log-probability of the action that was taken, the value estimate and the policy entropy (nats).
    -> dict(logp [n], values [n], entropy [n], logits [n,A])."""
    actions = np.ascontiguousarray(actions, dtype=np.int64)
    f = policy_forward(wt, obs)
    n = actions.shape[0]
    assert f["logits"].shape[0] == n and np.all((actions >= 0) & (actions < wt.A))
    logp, ent = np.empty(n), np.empty(n)
    for e in range(n):
        lp, h = log_softmax(f["logits"][e])
        logp[e], ent[e] = lp[actions[e]], h
    return {"logp": logp, "values": f["value"].copy(), "entropy": ent, "logits": f["logits"]}


def a2c_terms(logp, values, entropy, returns):
    """The three sample means the actor-critic update is built from (Section 3): the policy term of
    Eq. 4, (1/|D|) sum log pi(a_t|s_t) (R_t - V(s_t)), whose gradient with R_t - V held fixed is Eq. 4's first
    summand; the value loss J_V = (1/|D|) sum (R_t - V(s_t))^2; and the mean entropy that Eq. 4 weights by alpha.
    fp64 throughout.  -> (policy_term, value_loss, mean_entropy)."""
    logp, values, entropy, returns = (np.asarray(a, dtype=np.float64).ravel() for a in (logp, values, entropy, returns))
    count = logp.size
    assert count > 0 and values.size == count and entropy.size == count and returns.size == count
    pol = vl = ent = 0.0
    for i in range(count):
        adv = returns[i] - values[i]
        pol += logp[i] * adv
        vl += adv * adv
        ent += entropy[i]
    return pol / count, vl / count, ent / count


def delayed_update(theta, grad, sq_avg, lr: float, alpha: float, eps: float, precondition: bool = True):
    """One learner update of Section 4.1 "Delayed gradient", Eq. 5: theta_{j+1} = theta_j + eta * d, where the
    gradient of J-hat was taken at theta_{j-1} by the caller.  With RMSProp (Appendix F tables: momentum 0, epsilon
    given) d = g / (sqrt(v) + eps) and v <- alpha v + (1 - alpha) g^2 (Tieleman & Hinton's rule, denominator as in
    the table's epsilon); without it d = g.  fp64.  -> (theta_next, sq_avg_next)."""
    theta, grad, sq_avg = (np.asarray(a, dtype=np.float64) for a in (theta, grad, sq_avg))
    assert theta.shape == grad.shape == sq_avg.shape
    out_t, out_v = np.empty_like(theta), np.empty_like(sq_avg)
    ft, fg, fv, ot, ov = theta.ravel(), grad.ravel(), sq_avg.ravel(), out_t.ravel(), out_v.ravel()
    for i in range(ft.size):
        if precondition:
            v = alpha * fv[i] + (1.0 - alpha) * fg[i] * fg[i]
            d = fg[i] / (np.sqrt(v) + eps)
        else:
            v, d = fv[i], fg[i]
        ov[i] = v
        ot[i] = ft[i] + lr * d
    return out_t, out_v


def ppo_terms(logp_new, logp_old, values, entropy, advantages, returns, clip: float, normalize: bool):
    """Sample means of the clipped surrogate of proximal policy optimisation (Schulman et al. 2017, Eq. 7), the
    algorithm HTS-RL is run with on the football scenarios (Section 5, "Ours (PPO)"):
        rho_i = exp(logp_new_i - logp_old_i),   A_i the advantage (optionally standardised over the batch:
        (A - mean) / (std + 1e-8), population std),
        surrogate = mean(min(rho A, clip(rho, 1 - clip, 1 + clip) A)),
    plus the value loss mean((R - V)^2), the mean entropy and the fraction of samples with |rho - 1| > clip.
    fp64.  -> (surrogate, value_loss, mean_entropy, clip_fraction)."""
    lp, lo, v, h, a, r = (np.asarray(x, dtype=np.float64).ravel() for x in (logp_new, logp_old, values, entropy, advantages, returns))
    n = lp.size
    assert n > 0 and all(x.size == n for x in (lo, v, h, a, r)) and clip > 0
    if normalize:
        mean = 0.0
        for i in range(n):
            mean += a[i]
        mean /= n
        var = 0.0
        for i in range(n):
            var += (a[i] - mean) ** 2
        std = np.sqrt(var / n)
        a = (a - mean) / (std + 1e-8)
    sur = vl = ent = frac = 0.0
    for i in range(n):
        rho = np.exp(lp[i] - lo[i])
        clipped = min(max(rho, 1.0 - clip), 1.0 + clip)
        sur += min(rho * a[i], clipped * a[i])
        vl += (r[i] - v[i]) ** 2
        ent += h[i]
        frac += 1.0 if abs(rho - 1.0) > clip else 0.0
    return sur / n, vl / n, ent / n, frac / n


def vtrace(log_rhos, rewards, values, dones, bootstrap, gamma: float, lam: float, rho_bar: float, c_bar: float):
    """V-trace targets and truncated-importance-sampling policy-gradient advantages over a [T, N] storage: the
    off-policy correction of the systems the paper compares its delayed gradient with (Section 2, IMPALA;
    Appendix C, Table A1 "Truncated I.S."), taken from the cited paper's definition (Espeholt et al. 2018,
    Section 4.1, Eq. 1 and its Remark 1 recursion, and the policy-gradient term of Section 4.2):

        rho_t = min(rho_bar, pi/mu),   c_t = lam * min(c_bar, pi/mu),   pi/mu = exp(log_rhos_t)
        delta_t = rho_t (r_t + g_t V_{t+1} - V_t),          g_t = gamma (1 - d_t),  V_T = bootstrap
        vs_t - V_t = delta_t + g_t c_t (vs_{t+1} - V_{t+1}),   vs_T = bootstrap
        pg_t = rho_t (r_t + g_t vs_{t+1} - V_t)

    Plain backward loop in fp64; `dones` as in the advantage scan (a done cuts both the bootstrap and the trace).
    Returns (vs, pg_advantages) rounded to fp32.  Python loop over T, numpy over N."""
    lr, r, v, b = _f64(log_rhos), _f64(rewards), _f64(values), _f64(bootstrap)
    d = np.asarray(dones) != 0
    T, N = r.shape
    ratio = np.exp(lr)
    rho = np.minimum(float(rho_bar), ratio)
    c = float(lam) * np.minimum(float(c_bar), ratio)
    vs = np.empty((T, N), np.float64)
    pg = np.empty((T, N), np.float64)
    diff_next = np.zeros(N, np.float64)            # vs_{t+1} - V_{t+1}
    v_next = b.copy()
    vs_next = b.copy()
    for t in range(T - 1, -1, -1):
        g = float(gamma) * np.where(d[t], 0.0, 1.0)
        delta = rho[t] * (r[t] + g * v_next - v[t])
        diff = delta + g * c[t] * diff_next
        vs[t] = v[t] + diff
        pg[t] = rho[t] * (r[t] + g * vs_next - v[t])
        diff_next, v_next, vs_next = diff, v[t], vs[t]
    return vs.astype(np.float32), pg.astype(np.float32)


def objective(wt: Weights, obs, actions, advantages, returns, value_coef: float, entropy_coef: float,
              logp_old=None, clip: float = 0.0):
    """The scalar the learner ascends (Section 3, Eq. 4 is its gradient estimator; Eq. 5 applies that gradient):

        J-hat = (1/n) sum_i [ S_i - value_coef (R_i - V(s_i))^2 + entropy_coef H(pi(.|s_i)) ]

    with S_i = log pi(a_i|s_i) A_i for the actor-critic update (advantages held fixed: they are data), or, with
    `logp_old` and clip > 0, the clipped surrogate S_i = min(rho_i A_i, clip(rho_i, 1-clip, 1+clip) A_i),
    rho_i = exp(log pi(a_i|s_i) - logp_old_i), of the PPO runs.  fp64, from the forward oracle."""
    ev = evaluate_actions(wt, obs, actions)
    adv, ret = _f64(advantages).ravel(), _f64(returns).ravel()
    n = adv.size
    if logp_old is None or clip <= 0:
        s = ev["logp"] * adv
    else:
        rho = np.exp(ev["logp"] - _f64(logp_old).ravel())
        s = np.minimum(rho * adv, np.clip(rho, 1.0 - clip, 1.0 + clip) * adv)
    return float(np.sum(s - value_coef * (ret - ev["values"]) ** 2 + entropy_coef * ev["entropy"]) / n)


def _conv_backward(x, w, dy, stride):
    """Gradients of y[n,o,i,j] = b[o] + sum_{c,u,v} w[o,c,u,v] x[n,c,i s+u,j s+v] given dy: (dx, dw, db).
    One term of the chain rule per filter tap, written with strided views."""
    O, Cc, k, _ = w.shape
    _, _, Ho, Wo = dy.shape
    dx = np.zeros_like(x)
    dw = np.empty_like(w)
    for u in range(k):
        for v in range(k):
            xs = x[:, :, u:u + stride * Ho:stride, v:v + stride * Wo:stride]          # x[n,c,i s+u,j s+v]
            dw[:, :, u, v] = np.einsum("noij,ncij->oc", dy, xs)
            dx[:, :, u:u + stride * Ho:stride, v:v + stride * Wo:stride] += np.einsum("noij,oc->ncij", dy, w[:, :, u, v])
    return dx, dw, dy.sum(axis=(0, 2, 3))


def objective_grad(wt: Weights, obs, actions, advantages, returns, value_coef: float, entropy_coef: float,
                   logp_old=None, clip: float = 0.0):
    """Gradient of `objective` with respect to the twelve parameter tensors: the quantity Eq. 4 estimates and
    Eq. 5 adds to the parameters.  Chain rule through the network of Appendix F.1 / F.2 in fp64, layer by layer:
    heads (softmax and entropy derivatives in closed form), FC, the three convolutions; ReLU passes the gradient
    where its output is positive.  -> dict name -> array shaped like the parameter."""
    obs = np.ascontiguousarray(obs, dtype=np.uint8)
    n = obs.shape[0]
    f = policy_forward(wt, obs, taps=True)
    a = np.asarray(actions, dtype=np.int64)
    adv, ret = _f64(advantages).ravel(), _f64(returns).ravel()
    W = wt.arr
    logits, value = f["logits"], f["value"]
    m = logits.max(axis=1, keepdims=True)
    lse = m + np.log(np.exp(logits - m).sum(axis=1, keepdims=True))
    logp = logits - lse                                   # [n, A]
    p = np.exp(logp)
    ent = -(p * logp).sum(axis=1)
    onehot = np.zeros_like(p); onehot[np.arange(n), a] = 1.0
    lpa = logp[np.arange(n), a]
    # dS_i / dlogpi(a_i)
    if logp_old is None or clip <= 0:
        ds = adv.copy()
    else:
        rho = np.exp(lpa - _f64(logp_old).ravel())
        unclipped_active = rho * adv <= np.clip(rho, 1.0 - clip, 1.0 + clip) * adv      # the min takes the first argument
        ds = np.where(unclipped_active, rho * adv, 0.0)
    # d logpi(a) / d logit_j = [j == a] - p_j ;  dH / d logit_j = -p_j (log p_j + H)
    dlogits = (ds[:, None] * (onehot - p) - entropy_coef * p * (logp + ent[:, None])) / n
    dvalue = 2.0 * value_coef * (ret - value) / n
    g = {}
    h = f["fc"]                                           # [n, 512], after ReLU
    g["pi_w"] = dlogits.T @ h
    g["pi_b"] = dlogits.sum(axis=0)
    g["v_w"] = (dvalue[:, None] * h).sum(axis=0)[None, :]
    g["v_b"] = np.array([dvalue.sum()])
    dh = dlogits @ W["pi_w"] + dvalue[:, None] * W["v_w"]
    dh = dh * (h > 0)
    a3 = f["conv3"]
    flat = a3.reshape(n, -1)                              # (c, h, w) order, as the FC weight's columns
    g["fc_w"] = dh.T @ flat
    g["fc_b"] = dh.sum(axis=0)
    da3 = (dh @ W["fc_w"]).reshape(a3.shape) * (a3 > 0)
    a2, a1 = f["conv2"], f["conv1"]
    da2, g["conv3_w"], g["conv3_b"] = _conv_backward(a2, W["conv3_w"], da3, 1)
    da2 = da2 * (a2 > 0)
    da1, g["conv2_w"], g["conv2_b"] = _conv_backward(a1, W["conv2_w"], da2, 2)
    da1 = da1 * (a1 > 0)
    x = obs.astype(np.float64) / 255.0
    _, g["conv1_w"], g["conv1_b"] = _conv_backward(x, W["conv1_w"], da1, 4)
    return g
