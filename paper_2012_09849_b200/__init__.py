"""Python binding of the HTS-RL hot-path library (libhts.so, CUDA for sm_100a).

Argument marshalling only: every function here has the name and the meaning of the C
entry point it forwards to (see include/hts.h).  Tensors are ``torch`` CUDA tensors (torch is
used for device memory and streams, nothing else); the ``*_host`` calls take CPU tensors or
numpy arrays.  There is no fallback: if the library is missing or a call fails, an exception
is raised.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

from . import build as _build

HTS_OK = 0
HTS_DTYPE_FP32 = 0
HTS_DTYPE_BF16 = 1
STATUS_NAMES = ["HTS_OK", "HTS_ERR_INVALID_ARG", "HTS_ERR_SHAPE", "HTS_ERR_ALLOC", "HTS_ERR_CUDA",
                "HTS_ERR_TIMEOUT", "HTS_ERR_UNSUPPORTED"]
WEIGHT_NAMES = ("conv1_w", "conv1_b", "conv2_w", "conv2_b", "conv3_w", "conv3_b",
                "fc_w", "fc_b", "pi_w", "pi_b", "v_w", "v_b")
EXPORTS = ("hts_policy_create", "hts_policy_load_weights", "hts_policy_step", "hts_policy_step_indexed", "hts_policy_step_host",
           "hts_policy_evaluate", "hts_policy_gradient", "hts_a2c_terms", "hts_ppo_terms", "hts_delayed_update",
           "hts_policy_read_activation", "hts_action_uniforms", "hts_policy_profile", "hts_policy_profile_read",
           "hts_policy_kernel_name", "hts_last_async_error", "hts_policy_destroy", "hts_gae",
           "hts_gae_host", "hts_gae_host_release", "hts_vtrace", "hts_policy_step_noalloc", "hts_wait_selftest", "hts_launch_count", "hts_last_cuda_error", "hts_status_string")


class HtsError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        name = STATUS_NAMES[status] if 0 <= status < len(STATUS_NAMES) else str(status)
        detail = hts_last_cuda_error() if status == 4 else ""
        super().__init__(f"{what}: {name}" + (f" ({detail})" if detail else ""))


class hts_net_desc(C.Structure):
    _fields_ = [("C", C.c_int32), ("H", C.c_int32), ("W", C.c_int32), ("num_actions", C.c_int32),
                ("weight_dtype", C.c_int32), ("max_batch", C.c_int32)]


class hts_weights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in WEIGHT_NAMES]


class hts_grads(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in WEIGHT_NAMES]


_lib = None


def library_path() -> str:
    return _build.LIB


def lib():
    """Load libhts.so (built in-tree; see build.py).  Raises if it does not exist."""
    global _lib
    if _lib is None:
        path = library_path()
        if not os.path.exists(path):
            raise ImportError(f"{path} is missing: run `python -m paper_2012_09849_b200.build`")
        L = C.CDLL(path)
        vp, i32, u64, f32 = C.c_void_p, C.c_int32, C.c_uint64, C.c_float
        L.hts_policy_create.argtypes = [C.POINTER(hts_net_desc), C.POINTER(vp)]
        L.hts_policy_load_weights.argtypes = [vp, C.POINTER(hts_weights), vp]
        step = [vp, vp, vp, vp, i32, u64, i32, vp, vp, vp, vp, vp, vp]
        L.hts_policy_step.argtypes = step
        L.hts_policy_step_host.argtypes = step
        L.hts_policy_step_indexed.argtypes = [vp, vp, i32, vp, vp, vp, i32, u64, i32, vp, vp, vp, vp, vp]
        L.hts_policy_evaluate.argtypes = [vp, vp, vp, i32, vp, vp, vp, vp, vp]
        L.hts_policy_evaluate.restype = C.c_int
        L.hts_policy_gradient.argtypes = [vp, vp, vp, vp, vp, vp, f32, f32, f32, i32, C.POINTER(hts_grads), vp]
        L.hts_policy_gradient.restype = C.c_int
        L.hts_a2c_terms.argtypes = [vp, vp, vp, vp, C.c_int64, vp, vp]
        L.hts_a2c_terms.restype = C.c_int
        L.hts_ppo_terms.argtypes = [vp, vp, vp, vp, vp, vp, C.c_int64, f32, i32, vp, vp]
        L.hts_ppo_terms.restype = C.c_int
        L.hts_delayed_update.argtypes = [vp, vp, vp, C.c_int64, f32, f32, f32, vp, vp]
        L.hts_delayed_update.restype = C.c_int
        L.hts_policy_read_activation.argtypes = [vp, i32, i32, vp, vp]
        L.hts_action_uniforms.argtypes = [vp, vp, i32, u64, i32, i32, vp, vp]
        L.hts_policy_profile.argtypes = [vp, i32]
        L.hts_policy_profile.restype = C.c_int
        L.hts_policy_profile_read.argtypes = [vp, i32, C.POINTER(C.c_float), C.POINTER(i32)]
        L.hts_policy_profile_read.restype = C.c_int
        L.hts_policy_kernel_name.argtypes = [i32]
        L.hts_policy_kernel_name.restype = C.c_char_p
        L.hts_last_async_error.argtypes = [vp]
        L.hts_wait_selftest.argtypes = [vp, C.c_int64, vp]
        L.hts_wait_selftest.restype = C.c_int
        L.hts_policy_destroy.argtypes = [vp]
        L.hts_policy_destroy.restype = None
        gae = [vp, vp, vp, vp, f32, f32, i32, i32, vp, vp, vp]
        L.hts_gae.argtypes = gae
        L.hts_gae_host.argtypes = gae
        L.hts_vtrace.argtypes = [vp, vp, vp, vp, vp, f32, f32, f32, f32, i32, i32, vp, vp, vp]
        L.hts_vtrace.restype = C.c_int
        L.hts_gae_host_release.argtypes = []
        L.hts_gae_host_release.restype = C.c_int
        L.hts_policy_step_noalloc.argtypes = [C.POINTER(hts_net_desc), C.POINTER(hts_weights)] + step[1:]
        L.hts_policy_step_noalloc.restype = C.c_int
        L.hts_launch_count.restype = C.c_uint64
        L.hts_last_cuda_error.restype = C.c_char_p
        L.hts_status_string.restype = C.c_char_p
        L.hts_status_string.argtypes = [C.c_int]
        for name in ("hts_policy_create", "hts_policy_load_weights", "hts_policy_step", "hts_policy_step_indexed", "hts_policy_step_host",
                     "hts_policy_read_activation", "hts_action_uniforms", "hts_last_async_error", "hts_gae",
                     "hts_gae_host"):
            getattr(L, name).restype = C.c_int
        _lib = L
    return _lib


def _ptr(x):
    """Address of a torch tensor / numpy array / raw int / None."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if isinstance(x, np.ndarray):
        assert x.flags["C_CONTIGUOUS"]
        return x.ctypes.data
    assert x.is_contiguous()
    return x.data_ptr()


def _stream(stream):
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    return stream if isinstance(stream, int) else stream.cuda_stream


def _check(status: int, what: str):
    if status != HTS_OK:
        raise HtsError(status, what)


# ---- the entry points, one to one ---------------------------------------------------------
def hts_policy_create(C_: int, H: int, W: int, num_actions: int, weight_dtype: int, max_batch: int) -> int:
    d = hts_net_desc(C_, H, W, num_actions, weight_dtype, max_batch)
    out = C.c_void_p()
    _check(lib().hts_policy_create(C.byref(d), C.byref(out)), "hts_policy_create")
    return out.value


def hts_policy_load_weights(ctx: int, weights: dict, stream=None) -> None:
    """weights: name -> CUDA tensor (float32, or bfloat16 for a bf16 context), PyTorch layouts."""
    w = hts_weights(**{n: _ptr(weights[n]) for n in WEIGHT_NAMES})
    _check(lib().hts_policy_load_weights(ctx, C.byref(w), _stream(stream)), "hts_policy_load_weights")


def hts_policy_step(ctx, obs, env_ids, t_per_env, t, seed, n, actions, logp, values, entropy,
                    logits=None, stream=None) -> None:
    _check(lib().hts_policy_step(ctx, _ptr(obs), _ptr(env_ids), _ptr(t_per_env), int(t), int(seed), int(n),
                                 _ptr(actions), _ptr(logp), _ptr(values), _ptr(entropy), _ptr(logits),
                                 _stream(stream)), "hts_policy_step")


def hts_policy_step_indexed(ctx, state_buffer, pool, slots, env_ids, t_per_env, t, seed, n, actions_row, logp_row,
                            values_row, entropy_row, stream=None) -> None:
    _check(lib().hts_policy_step_indexed(ctx, _ptr(state_buffer), int(pool), _ptr(slots), _ptr(env_ids), _ptr(t_per_env),
                                         int(t), int(seed), int(n), _ptr(actions_row), _ptr(logp_row), _ptr(values_row),
                                         _ptr(entropy_row), _stream(stream)), "hts_policy_step_indexed")


def hts_policy_evaluate(ctx, obs, actions, n, logp, values, entropy, logits=None, stream=None) -> None:
    _check(lib().hts_policy_evaluate(ctx, _ptr(obs), _ptr(actions), int(n), _ptr(logp), _ptr(values), _ptr(entropy),
                                     _ptr(logits), _stream(stream)), "hts_policy_evaluate")


def hts_policy_gradient(ctx, obs, actions, advantages, returns, logp_old, value_coef, entropy_coef, clip, n, grads: dict,
                        stream=None) -> None:
    """grads: name -> CUDA float32 tensor shaped like the parameter (overwritten)."""
    g = hts_grads(**{k: _ptr(grads[k]) for k in WEIGHT_NAMES})
    _check(lib().hts_policy_gradient(ctx, _ptr(obs), _ptr(actions), _ptr(advantages), _ptr(returns), _ptr(logp_old),
                                     float(value_coef), float(entropy_coef), float(clip), int(n), C.byref(g),
                                     _stream(stream)), "hts_policy_gradient")


def hts_a2c_terms(logp, values, entropy, returns, count, out3, stream=None) -> None:
    _check(lib().hts_a2c_terms(_ptr(logp), _ptr(values), _ptr(entropy), _ptr(returns), int(count), _ptr(out3),
                               _stream(stream)), "hts_a2c_terms")


def hts_ppo_terms(logp_new, logp_old, values, entropy, advantages, returns, count, clip, normalize, out4, stream=None) -> None:
    _check(lib().hts_ppo_terms(_ptr(logp_new), _ptr(logp_old), _ptr(values), _ptr(entropy), _ptr(advantages), _ptr(returns),
                               int(count), float(clip), int(bool(normalize)), _ptr(out4), _stream(stream)), "hts_ppo_terms")


def hts_delayed_update(theta, grad, sq_avg, count, lr, alpha, eps, theta_bf16=None, stream=None) -> None:
    _check(lib().hts_delayed_update(_ptr(theta), _ptr(grad), _ptr(sq_avg), int(count), float(lr), float(alpha), float(eps),
                                    _ptr(theta_bf16), _stream(stream)), "hts_delayed_update")


def hts_policy_step_host(ctx, obs, env_ids, t_per_env, t, seed, n, actions, logp, values, entropy,
                         logits=None, stream=None) -> None:
    _check(lib().hts_policy_step_host(ctx, _ptr(obs), _ptr(env_ids), _ptr(t_per_env), int(t), int(seed), int(n),
                                      _ptr(actions), _ptr(logp), _ptr(values), _ptr(entropy), _ptr(logits),
                                      _stream(stream)), "hts_policy_step_host")


def hts_policy_read_activation(ctx, layer: int, n: int, out, stream=None) -> None:
    _check(lib().hts_policy_read_activation(ctx, int(layer), int(n), _ptr(out), _stream(stream)),
           "hts_policy_read_activation")


def hts_action_uniforms(env_ids, t_per_env, t, seed, n, num_actions, out, stream=None) -> None:
    _check(lib().hts_action_uniforms(_ptr(env_ids), _ptr(t_per_env), int(t), int(seed), int(n), int(num_actions),
                                     _ptr(out), _stream(stream)), "hts_action_uniforms")


def hts_policy_profile(ctx, enable: bool) -> None:
    _check(lib().hts_policy_profile(ctx, int(bool(enable))), "hts_policy_profile")


def hts_policy_profile_read(ctx, kernel: int):
    """-> (total milliseconds, launches) of one kernel of the actor step since profiling was enabled."""
    ms, cnt = C.c_float(), C.c_int32()
    _check(lib().hts_policy_profile_read(ctx, int(kernel), C.byref(ms), C.byref(cnt)), "hts_policy_profile_read")
    return ms.value, cnt.value


def hts_policy_kernel_name(kernel: int) -> str:
    return lib().hts_policy_kernel_name(int(kernel)).decode()


def hts_last_async_error(ctx) -> int:
    return int(lib().hts_last_async_error(ctx))


def hts_wait_selftest(ctx, limit_ticks: int, stream=None) -> None:
    _check(lib().hts_wait_selftest(ctx, int(limit_ticks), _stream(stream)), "hts_wait_selftest")


def hts_policy_destroy(ctx) -> None:
    lib().hts_policy_destroy(ctx)


def hts_gae(rewards, values, dones, bootstrap, gamma, lam, T, N, advantages, returns, stream=None) -> None:
    _check(lib().hts_gae(_ptr(rewards), _ptr(values), _ptr(dones), _ptr(bootstrap), float(gamma), float(lam),
                         int(T), int(N), _ptr(advantages), _ptr(returns), _stream(stream)), "hts_gae")


def hts_gae_host(rewards, values, dones, bootstrap, gamma, lam, T, N, advantages, returns, stream=None) -> None:
    _check(lib().hts_gae_host(_ptr(rewards), _ptr(values), _ptr(dones), _ptr(bootstrap), float(gamma), float(lam),
                              int(T), int(N), _ptr(advantages), _ptr(returns), _stream(stream)), "hts_gae_host")


def hts_vtrace(log_rhos, rewards, values, dones, bootstrap, gamma, lam, rho_bar, c_bar, T, N, vs, pg_advantages,
               stream=None) -> None:
    _check(lib().hts_vtrace(_ptr(log_rhos), _ptr(rewards), _ptr(values), _ptr(dones), _ptr(bootstrap), float(gamma),
                            float(lam), float(rho_bar), float(c_bar), int(T), int(N), _ptr(vs), _ptr(pg_advantages),
                            _stream(stream)), "hts_vtrace")


def hts_gae_host_release() -> None:
    _check(lib().hts_gae_host_release(), "hts_gae_host_release")


def hts_policy_step_noalloc(C_, H, W, num_actions, weights: dict, obs, env_ids, t_per_env, t, seed, n,
                            actions, logp, values, entropy, logits=None, stream=None) -> None:
    """Actor step without any allocation: fp32 weights (dict of CUDA float32 tensors) are read in place and
    the hidden activations use the library's fixed 4 MiB scratch array (see hts.h for the limits)."""
    d = hts_net_desc(C_, H, W, num_actions, HTS_DTYPE_FP32, n)
    w = hts_weights(**{k: _ptr(weights[k]) for k in WEIGHT_NAMES})
    _check(lib().hts_policy_step_noalloc(C.byref(d), C.byref(w), _ptr(obs), _ptr(env_ids), _ptr(t_per_env), int(t),
                                         int(seed), int(n), _ptr(actions), _ptr(logp), _ptr(values), _ptr(entropy),
                                         _ptr(logits), _stream(stream)), "hts_policy_step_noalloc")


def hts_launch_count() -> int:
    return int(lib().hts_launch_count())


def hts_last_cuda_error() -> str:
    return lib().hts_last_cuda_error().decode()


def hts_status_string(status: int) -> str:
    return lib().hts_status_string(int(status)).decode()


# ---- marshalling helper for weights --------------------------------------------------------
def weights_to_device(params: dict, weight_dtype: int, device="cuda"):
    """numpy fp32 parameter dict -> dict of CUDA tensors in the context's weight dtype."""
    import torch
    dt = torch.float32 if weight_dtype == HTS_DTYPE_FP32 else torch.bfloat16
    return {k: torch.from_numpy(np.ascontiguousarray(params[k], dtype=np.float32)).to(device).to(dt).contiguous()
            for k in WEIGHT_NAMES}
