#!/usr/bin/env python
"""Benchmark of the HTS-RL hot path on B200: actor env-steps/s over whole rollouts.

One step = one rollout of the "ppo_atari_large" workload: T=128 batched actor steps over
N=1024 environments (uint8 4x84x84 observations from a ring of pre-generated batches larger
than L2) writing values/log-probs/actions into one of two rollout storages, plus the GAE scan
of the previous rollout on a second stream (its bootstrap is the value row 0 of the rollout
being collected), as in the paper's concurrent rollout and learning.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints one JSON line (rank 0).  With N > 1 (torchrun) every rank runs the same workload on
its own range of environment ids; there is no data-path collective.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import hts_workloads as wl  # noqa: E402

WORKLOAD = 3                       # hts_workloads.CONFIGS index
# dram__bytes_read.sum + dram__bytes_write.sum of one launch of a kernel at this workload (n = 1024), from one ncu
# capture of that kernel; None once the kernel has changed since its counters were taken
DRAM_TRAFFIC_BYTES = {"conv1": 28953344 + 242432, "conv2": None, "conv3": None, "fc": None, "heads": None}
DTYPE = "bf16 weights, fp16 operands, fp32 accumulate"
METRIC = "actor env-steps/s (whole rollout: T actor steps + GAE)"
UNIT = "env-steps/s"
SEED = 0x5EED


def macs_per_env_step(cfg) -> int:
    h1, w1 = wl.conv_out(cfg.H, 8, 4), wl.conv_out(cfg.W, 8, 4)
    h2, w2 = wl.conv_out(h1, 4, 2), wl.conv_out(w1, 4, 2)
    h3, w3 = wl.conv_out(h2, 3, 1), wl.conv_out(w2, 3, 1)
    return (32 * h1 * w1 * cfg.C * 64 + 64 * h2 * w2 * 32 * 16 + 64 * h3 * w3 * 64 * 9
            + 512 * 64 * h3 * w3 + (cfg.A + 1) * 512)


def layer_macs(cfg) -> dict:
    h1, w1 = wl.conv_out(cfg.H, 8, 4), wl.conv_out(cfg.W, 8, 4)
    h2, w2 = wl.conv_out(h1, 4, 2), wl.conv_out(w1, 4, 2)
    h3, w3 = wl.conv_out(h2, 3, 1), wl.conv_out(w2, 3, 1)
    return {"conv1": 32 * h1 * w1 * cfg.C * 64, "conv2": 64 * h2 * w2 * 32 * 16,
            "conv3": 64 * h3 * w3 * 64 * 9, "fc": 512 * 64 * h3 * w3, "heads": (cfg.A + 1) * 512}


def measured_peaks() -> tuple[dict, str]:
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.rows, self.proc, self.index = [], None, index

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                 "-lms", "20"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except (ValueError, IndexError):
                continue
            for name, val in zip(names, r[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        busy = sorted(sm)[len(sm) // 2:] if sm else []           # upper half: samples under load
        return {"sm_mhz": float(np.median(busy)) if busy else None,
                "sm_max_mhz": max(mx) if mx else None, "reasons": sorted(reasons), "samples": len(sm)}


# ------------------------------------------------------------------------------------------------
def run_reference(args) -> None:
    """The CPU oracle as it stands, on a bounded sample per step, on this host's cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import hts_oracle as orc
    cfg = wl.CONFIGS[WORKLOAD]
    wt = orc.Weights(wl.make_weights(cfg))
    r, v, d, b = wl.make_rollout(cfg)
    sample_rows = 512
    env_ids = np.arange(sample_rows, dtype=np.int32)
    obs = [wl.make_obs(cfg, sample_rows, batch_index=i) for i in range(2)]

    def one(i):
        t0 = time.perf_counter()
        orc.policy_step(wt, obs[i % 2], env_ids, i, SEED)
        t1 = time.perf_counter()
        orc.gae(r, v, d, b, cfg.gamma, cfg.lam)
        t2 = time.perf_counter()
        return t1 - t0, t2 - t1

    for i in range(args.warmup):
        one(i)
    ta = tg = 0.0
    for i in range(args.steps):
        a, g = one(i)
        ta += a; tg += g
    per_env_step = ta / (args.steps * sample_rows) + tg / (args.steps * cfg.T * cfg.N)
    value = 1.0 / per_env_step
    sample = (f"per step: one actor step on {sample_rows} of {cfg.N} envs + one full GAE [{cfg.T},{cfg.N}]; "
              f"rate = 1/(actor s per env-step + GAE s per element)")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * (ta + tg) / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": cfg.name, "N": cfg.N, "T": cfg.T, "obs": [cfg.C, cfg.H, cfg.W], "actions": cfg.A},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": orc.num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


# ------------------------------------------------------------------------------------------------
def run_ncu_case(steps: int, rows: int = 0) -> None:
    """A few actor steps of the bench workload (n = N rows each, or `rows` of the same frames and network) and
    one GAE over [T, N]: the small case that is captured under ncu.  Device footprint: two observation batches
    and the context (< 0.2 GB at 1024 rows, < 1 GB at 8192)."""
    import torch
    import paper_2012_09849_b200 as hts
    cfg = wl.CONFIGS[WORKLOAD]
    T, N = cfg.T, (rows if rows > 0 else cfg.N)
    ctx = hts.hts_policy_create(cfg.C, cfg.H, cfg.W, cfg.A, hts.HTS_DTYPE_BF16, N)
    hts.hts_policy_load_weights(ctx, hts.weights_to_device(wl.make_weights(cfg), hts.HTS_DTYPE_BF16))
    obs = [torch.from_numpy(wl.make_obs(cfg, N, batch_index=i)).cuda() for i in range(2)]
    ids = torch.arange(N, dtype=torch.int32, device="cuda")
    act = torch.empty(N, dtype=torch.int32, device="cuda")
    f = [torch.empty(N, device="cuda") for _ in range(3)]
    for t in range(steps):
        hts.hts_policy_step(ctx, obs[t % 2], ids, None, t, SEED, N, act, *f)
    r, v, d, b = (torch.from_numpy(x).cuda() for x in wl.make_rollout(cfg, T=T, N=N))
    adv, ret = torch.empty_like(v), torch.empty_like(v)
    hts.hts_gae(r, v, d, b, cfg.gamma, cfg.lam, T, N, adv, ret)
    torch.cuda.synchronize()
    hts.hts_policy_destroy(ctx)
    print("ncu case done:", steps, "steps")


# ------------------------------------------------------------------------------------------------
def run_ncu_learner_case() -> None:
    """The HBM-bound kernels on a shape larger than L2 but small enough to capture (2^25 transitions, 134 MB per
    array, under 1.5 GB on the device): the advantage scan, both sample-mean kernels and the parameter update,
    launched twice each (the second launch is the one to capture)."""
    import torch
    import paper_2012_09849_b200 as hts
    cfg = wl.CONFIGS[WORKLOAD]
    T, N = cfg.T, (1 << 25) // cfg.T
    r, v, d, b = (torch.from_numpy(x).cuda() for x in wl.make_rollout(cfg, T=T, N=N))
    adv, ret = torch.empty_like(v), torch.empty_like(v)
    lp_new, lp_old = -torch.rand_like(v), -torch.rand_like(v)
    out = torch.empty(4, device="cuda")
    half = torch.empty(T * N, dtype=torch.bfloat16, device="cuda")
    for _ in range(2):
        hts.hts_gae(r, v, d, b, cfg.gamma, cfg.lam, T, N, adv, ret)
        hts.hts_a2c_terms(lp_new, v, lp_old, ret, T * N, out)
        hts.hts_ppo_terms(lp_new, lp_old, v, r, adv, ret, T * N, 0.2, True, out)
        hts.hts_delayed_update(lp_new, adv, lp_old.abs_(), T * N, 7e-4, 0.99, 1e-5, half)
    torch.cuda.synchronize()
    print("ncu learner case done:", T * N, "transitions")


# ------------------------------------------------------------------------------------------------
def run_batch_sweep() -> None:
    """Actor-step time against the executor batch size, 1..8192 rows of the 8192-environment pool of the
    asynchronous-executor configuration (4x84x84 frames, 18 actions); prints a markdown table."""
    import torch
    import paper_2012_09849_b200 as hts
    cfg = wl.CONFIGS[5]
    pool = cfg.N
    ctx = hts.hts_policy_create(cfg.C, cfg.H, cfg.W, cfg.A, hts.HTS_DTYPE_BF16, pool)
    hts.hts_policy_load_weights(ctx, hts.weights_to_device(wl.make_weights(cfg), hts.HTS_DTYPE_BF16))
    obs = [torch.from_numpy(wl.make_obs(cfg, pool, batch_index=i)).cuda() for i in range(2)]
    ids = torch.arange(pool, dtype=torch.int32, device="cuda")
    act = torch.empty(pool, dtype=torch.int32, device="cuda")
    f = [torch.empty(pool, device="cuda") for _ in range(3)]
    macs = macs_per_env_step(cfg)
    print("| batch n | us per step | env-steps/s | TFLOP/s |")
    print("|---|---|---|---|")
    n = 1
    while n <= pool:
        reps = 50 if n <= 1024 else 20
        for t in range(5):
            hts.hts_policy_step(ctx, obs[t % 2], ids, None, t, SEED, n, act, *f)
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for t in range(reps):
            hts.hts_policy_step(ctx, obs[t % 2], ids, None, t, SEED, n, act, *f)
        b.record(); torch.cuda.synchronize()
        us = 1e3 * a.elapsed_time(b) / reps
        print(f"| {n} | {us:.1f} | {n / us * 1e6:.3g} | {2 * macs * n / us / 1e6:.1f} |", flush=True)
        n *= 2
    hts.hts_policy_destroy(ctx)


# ------------------------------------------------------------------------------------------------
def config_points(hts, torch, dev, peaks, stream, l2_bytes) -> dict:
    """The other configurations on the same line: actor-step time at the configuration's own batch (frames from a
    ring of device-generated batches larger than twice L2, same value law as the seeded recipe) and the advantage
    scan at its own [T, N] with L2 flushed between launches."""
    out = {}
    flush = torch.empty(2 * l2_bytes, dtype=torch.uint8, device=dev)
    for ci in (1, 2, 4):
        c = wl.CONFIGS[ci]
        n = c.N
        dt = hts.HTS_DTYPE_FP32 if c.weight_dtype == "fp32" else hts.HTS_DTYPE_BF16
        ctx = hts.hts_policy_create(c.C, c.H, c.W, c.A, dt, n)
        hts.hts_policy_load_weights(ctx, hts.weights_to_device(wl.make_weights(c), dt, dev))
        per_batch = n * c.C * c.H * c.W
        ring = max(4, -(-2 * l2_bytes // per_batch))
        g = torch.Generator(device=dev); g.manual_seed(1000 + ci)
        if c.obs_law == "uniform":
            frames = torch.randint(0, 256, (ring, n, c.C, c.H, c.W), dtype=torch.uint8, device=dev, generator=g)
        else:
            frames = ((torch.rand((ring, n, c.C, c.H, c.W), device=dev, generator=g) < 0.02) * 255).to(torch.uint8)
        p_fr = [frames[i].data_ptr() for i in range(ring)]
        ids = torch.arange(n, dtype=torch.int32, device=dev)
        o = [torch.empty(n, dtype=torch.int32, device=dev)] + [torch.empty(n, device=dev) for _ in range(3)]
        reps = 200 if n <= 256 else 100
        for t in range(10):
            hts.hts_policy_step(ctx, p_fr[t % ring], ids, None, t, SEED, n, *o, None, stream.cuda_stream)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for t in range(reps):
            hts.hts_policy_step(ctx, p_fr[t % ring], ids, None, t, SEED, n, *o, None, stream.cuda_stream)
        b.record(stream); torch.cuda.synchronize()
        us = 1e3 * a.elapsed_time(b) / reps
        hts.hts_policy_destroy(ctx)
        del frames
        tf = 2.0 * macs_per_env_step(c) * n / (us * 1e-6) / 1e12
        weight_bytes = (2 if dt == hts.HTS_DTYPE_BF16 else 4) * sum(int(np.prod(v.shape)) for v in wl.make_weights(c).values())
        # the advantage scan at the configuration's own size, cold
        r, v, d, bt = (torch.from_numpy(x).to(dev) for x in wl.make_rollout(c))
        adv, ret = torch.empty_like(v), torch.empty_like(v)
        g_ms = []
        for i in range(12):
            with torch.cuda.stream(stream):
                flush.fill_(i)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            hts.hts_gae(r, v, d, bt, c.gamma, c.lam, c.T, c.N, adv, ret, stream)
            b.record(stream); torch.cuda.synchronize()
            g_ms.append(a.elapsed_time(b))
        gae_us = 1e3 * float(np.median(g_ms[3:]))
        out[f"cfg{ci}"] = {
            "workload": c.name, "n": n, "obs": [c.C, c.H, c.W], "weights": c.weight_dtype, "ring_batches": ring,
            "actor_step_us": us, "env_steps_per_s": n / (us * 1e-6), "tflops": tf,
            "frac_of_bf16_burst": tf / peaks["bf16_tflops"], "frac_of_bf16_sustained": tf / peaks["bf16_tflops_sustained"],
            "hbm_gbs_over_frames_and_weights": (per_batch + weight_bytes) / (us * 1e-6) / 1e9,
            "gae": {"T": c.T, "N": c.N, "us_cold": gae_us, "elems_per_s": c.T * c.N / (gae_us * 1e-6),
                    "gbs_cold": (17 * c.T * c.N + 4 * c.N) / (gae_us * 1e-6) / 1e9}}
    return out


# ------------------------------------------------------------------------------------------------
def run_ours(args) -> None:
    import torch
    import paper_2012_09849_b200 as hts

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    cfg = wl.CONFIGS[WORKLOAD]
    T, N, A = cfg.T, cfg.N, cfg.A
    obs_bytes = cfg.C * cfg.H * cfg.W
    peaks, peak_kind = measured_peaks()
    l2 = torch.cuda.get_device_properties(local).L2_cache_size
    ring = max(8, -(-2 * l2 // (N * obs_bytes)))                 # ring of distinct batches > 2x L2
    dev = torch.device("cuda", local)

    ctx = hts.hts_policy_create(cfg.C, cfg.H, cfg.W, A, hts.HTS_DTYPE_BF16, N)
    params = wl.make_weights(cfg)
    dev_w = hts.weights_to_device(params, hts.HTS_DTYPE_BF16, dev)
    hts.hts_policy_load_weights(ctx, dev_w)
    obs_host = [torch.from_numpy(wl.make_obs(cfg, N, batch_index=i)).pin_memory() for i in range(ring)]
    obs_dev = [o.to(dev) for o in obs_host]
    lo, hi = rank_env_range(rank, N)
    env_ids = torch.arange(lo, hi, dtype=torch.int32, device=dev)
    r_np, _, d_np, _ = wl.make_rollout(cfg)
    rewards, dones = torch.from_numpy(r_np).to(dev), torch.from_numpy(d_np).to(dev)

    from paper_2012_09849_b200.pipeline import RolloutPipeline
    p_obs = [o.data_ptr() for o in obs_dev]
    pipe = RolloutPipeline(ctx, T, N, env_ids, rewards, dones, cfg.gamma, cfg.lam,
                           obs_for=lambda k, t: p_obs[(k * T + t) % ring], seed_for=lambda k: SEED + k, device=dev)
    store, s_act, s_gae = pipe.store, pipe.s_act, pipe.s_gae
    rollout = pipe.rollout
    p_ids, h_act_stream, h_gae_stream = env_ids.data_ptr(), s_act.cuda_stream, s_gae.cuda_stream

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    rollout(-1)                                                  # fills storage 1 so the first GAE has input
    for k in range(args.warmup):
        rollout(k)
    barrier()

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    launches0 = hts.hts_launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(s_act)
    for k in range(args.steps):
        rollout(args.warmup + k)
    pipe.join()
    e1.record(s_act)
    barrier()
    launches = hts.hts_launch_count() - launches0
    clocks = sampler.stop() if rank == 0 else None
    ms = e0.elapsed_time(e1)
    if dist is not None:
        tms = torch.tensor([ms], device=dev); dist.all_reduce(tms, op=dist.ReduceOp.MAX); ms = float(tms.item())
    value = world * args.steps * T * N / (ms * 1e-3)

    # ---- per-kernel device times over the same region (second pass, events around each kernel)
    hts.hts_policy_profile(ctx, True)
    for k in range(min(args.steps, 4096 // T)):
        rollout(args.warmup + args.steps + k)
    torch.cuda.synchronize()
    hts.hts_policy_profile(ctx, False)
    kern = {}
    for i in range(5):
        tot, cnt = hts.hts_policy_profile_read(ctx, i)
        kern[hts.hts_policy_kernel_name(i)] = {"ms_total": tot, "launches": cnt,
                                               "us_per_launch": 1e3 * tot / max(cnt, 1)}
    # GAE alone, cold (inputs evicted by a write larger than L2 between launches)
    flush = torch.empty(2 * l2, dtype=torch.uint8, device=dev)
    g_ms = []
    for i in range(20):
        with torch.cuda.stream(s_gae):
            flush.fill_(i)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(s_gae)
        hts.hts_gae(rewards, store[0].values, dones, store[1].values[0], cfg.gamma, cfg.lam, T, N,
                    store[0].adv, store[0].ret, s_gae)
        b.record(s_gae); torch.cuda.synchronize()
        g_ms.append(a.elapsed_time(b))
    gae_us = 1e3 * float(np.median(g_ms[3:]))
    gae_bytes = 17 * T * N + 4 * N
    # GAE on a widened shape (same T and laws, N = 2^20): the kernel's HBM asymptote
    Nw = 1 << 20
    rw, vw, dw, bw = (torch.from_numpy(x).to(dev) for x in wl.make_rollout(cfg, T=T, N=Nw))
    aw, qw = torch.empty_like(vw), torch.empty_like(vw)
    w_ms = []
    for i in range(8):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(s_gae)
        hts.hts_gae(rw, vw, dw, bw, cfg.gamma, cfg.lam, T, Nw, aw, qw, s_gae)
        b.record(s_gae); torch.cuda.synchronize()
        w_ms.append(a.elapsed_time(b))
    wide_ms = float(np.median(w_ms[3:]))
    wide_gbs = (17 * T * Nw + 4 * Nw) / (wide_ms * 1e-3) / 1e9
    # the off-policy-corrected scan (V-trace / truncated importance sampling) on the same widened shape: 21 bytes per element
    lw = torch.zeros_like(vw).uniform_(-0.5, 0.5)
    pw = torch.empty_like(vw)
    v_ms = []
    for i in range(8):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(s_gae)
        hts.hts_vtrace(lw, rw, vw, dw, bw, cfg.gamma, cfg.lam, 1.0, 1.0, T, Nw, aw, pw, s_gae)
        b.record(s_gae); torch.cuda.synchronize()
        v_ms.append(a.elapsed_time(b))
    vtrace_ms = float(np.median(v_ms[3:]))
    vtrace_gbs = (21 * T * Nw + 4 * Nw) / (vtrace_ms * 1e-3) / 1e9
    del lw, pw
    # the learner's sample means (policy term of Eq. 4, value loss, entropy) over the same widened storage
    # (16 bytes per transition) and over the configuration's own [T, N] storage
    out3 = torch.empty(3, dtype=torch.float32, device=dev)
    t_ms = []
    for i in range(8):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(s_gae)
        hts.hts_a2c_terms(aw, vw, rw, qw, T * Nw, out3, s_gae)
        b.record(s_gae); torch.cuda.synchronize()
        t_ms.append(a.elapsed_time(b))
    terms_wide_ms = float(np.median(t_ms[3:]))
    terms_wide_gbs = 16 * T * Nw / (terms_wide_ms * 1e-3) / 1e9
    t_ms = []
    for i in range(12):
        with torch.cuda.stream(s_gae):
            flush.fill_(i)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(s_gae)
        hts.hts_a2c_terms(store[0].logp, store[0].values, store[0].entropy, store[0].ret, T * N, out3, s_gae)
        b.record(s_gae); torch.cuda.synchronize()
        t_ms.append(a.elapsed_time(b))
    terms_us = 1e3 * float(np.median(t_ms[3:]))
    # the PPO form (clipped surrogate, standardised advantages: two passes over the advantages + one over all six arrays)
    out4 = torch.empty(4, dtype=torch.float32, device=dev)
    x1, x2 = torch.zeros_like(vw), torch.zeros_like(vw)          # six distinct arrays
    t_ms = []
    for i in range(8):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(s_gae)
        hts.hts_ppo_terms(aw, x1, vw, qw, rw, x2, T * Nw, 0.2, True, out4, s_gae)
        b.record(s_gae); torch.cuda.synchronize()
        t_ms.append(a.elapsed_time(b))
    ppo_wide_ms = float(np.median(t_ms[3:]))
    ppo_wide_gbs = 32 * T * Nw / (ppo_wide_ms * 1e-3) / 1e9
    del x1, x2
    # the learner's parameter update (Eq. 5 with RMSProp scaling) over a parameter vector of the widened size
    upd_ms = []
    hb = torch.empty(T * Nw, dtype=torch.bfloat16, device=dev)
    aw.zero_(); qw.fill_(1e-4)
    for i in range(8):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(s_gae)
        hts.hts_delayed_update(aw, vw, qw, T * Nw, 7e-4, 0.99, 1e-5, hb, s_gae)
        b.record(s_gae); torch.cuda.synchronize()
        upd_ms.append(a.elapsed_time(b))
    upd_wide_ms = float(np.median(upd_ms[3:]))
    upd_gbs = 22 * T * Nw / (upd_wide_ms * 1e-3) / 1e9
    del hb

    # ---- dominant kernel and its roofline (both the burst and the sustained measured peaks)
    macs = layer_macs(cfg)
    top = max(kern, key=lambda k: kern[k]["ms_total"])
    top_us = kern[top]["us_per_launch"]
    achieved_tf = 2.0 * macs[top] * N / (top_us * 1e-6) / 1e12
    peak_tf, peak_burst = peaks["bf16_tflops_sustained"], peaks["bf16_tflops"]
    roofline = {"bound": "tensor", "kernel": top, "achieved": achieved_tf, "peak": peak_burst, "unit": "TFLOP/s",
                "frac": achieved_tf / peak_burst, "frac_burst": achieved_tf / peak_burst,
                "frac_sustained": achieved_tf / peak_tf, "peak_sustained": peak_tf,
                "peak_kind": peak_kind + " burst (the timed region is a fraction of a second at full clocks)",
                "traffic": DRAM_TRAFFIC_BYTES.get(top),
                "algorithmic_bytes": N * obs_bytes if top == "conv1" else None,
                "us_per_launch": top_us}
    for name, kk in kern.items():
        tf = 2.0 * macs[name] * N / (max(kk["us_per_launch"], 1e-9) * 1e-6) / 1e12
        kk["tflops"] = tf
        kk["frac_burst"] = tf / peak_burst
    whole_tf = 2.0 * macs_per_env_step(cfg) * value / world / 1e12

    # ---- overlap of the two streams: one rollout of actor steps and the advantage scan of the widened storage
    #      (long enough to matter), run one after the other on one stream and side by side on two
    def timed(fn, reps=3):
        ms = []
        for _ in range(reps):
            torch.cuda.synchronize()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(s_act)
            fn()
            b.record(s_act); torch.cuda.synchronize()
            ms.append(a.elapsed_time(b))
        return float(np.median(ms))

    def actor_only():
        for t in range(T):
            hts.hts_policy_step(ctx, p_obs[t % ring], p_ids, None, t, SEED, N, store[0].p_act[t], store[0].p_logp[t],
                                store[0].p_val[t], store[0].p_ent[t], None, h_act_stream)

    def gae_wide(stream_handle):
        hts.hts_gae(rw, vw, dw, bw, cfg.gamma, cfg.lam, T, Nw, aw, qw, stream_handle)

    def serial():
        actor_only(); gae_wide(h_act_stream)

    def overlapped():
        s_gae.wait_stream(s_act)
        gae_wide(h_gae_stream)
        actor_only()
        s_act.wait_stream(s_gae)

    # host time to enqueue one actor step: a burst short enough not to fill the launch queue (a full queue makes
    # the host wait for the GPU and the two times look alike), started on an idle device
    torch.cuda.synchronize()
    burst = 48
    host_t0 = time.perf_counter()
    for t in range(burst):
        hts.hts_policy_step(ctx, p_obs[t % ring], p_ids, None, t, SEED, N, store[0].p_act[t], store[0].p_logp[t],
                            store[0].p_val[t], store[0].p_ent[t], None, h_act_stream)
    host_enqueue_us = 1e6 * (time.perf_counter() - host_t0) / burst
    torch.cuda.synchronize()

    overlap = {"actor_ms": timed(actor_only), "gae_ms": timed(lambda: gae_wide(h_act_stream)),
               "serial_ms": timed(serial), "overlapped_ms": timed(overlapped),
               "what": f"{T} actor steps of {N} rows and one advantage scan over [{T},{Nw}]"}
    del rw, vw, dw, bw, aw, qw

    # ---- the executor-facing form: frames gathered by slot from a state buffer (one ring entry), outputs
    #      scattered to the same slots of a storage row; slots = a random permutation of the pool
    perm = torch.from_numpy(np.random.default_rng(SEED).permutation(N).astype(np.int32)).to(dev)
    p_perm = perm.data_ptr()
    st0 = store[0]

    def indexed_steps(count):
        for t in range(count):
            hts.hts_policy_step_indexed(ctx, p_obs[t % ring], N, p_perm, p_ids, None, t % T, SEED, N,
                                        st0.p_act[t % T], st0.p_logp[t % T], st0.p_val[t % T], st0.p_ent[t % T],
                                        h_act_stream)
    indexed_steps(8)
    torch.cuda.synchronize()
    i0, i1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    i0.record(s_act)
    indexed_steps(2 * T)
    i1.record(s_act); torch.cuda.synchronize()
    indexed_us = 1e3 * i0.elapsed_time(i1) / (2 * T)

    # ---- end to end through the host-buffer entry points
    if rank == 0 or dist is not None:
        h_act = torch.empty(T, N, dtype=torch.int32).pin_memory()
        h_logp, h_val, h_ent, h_adv, h_ret = (torch.empty(T, N, dtype=torch.float32).pin_memory() for _ in range(5))
        h_ids = env_ids.cpu().pin_memory()
        h_rew, h_done = torch.from_numpy(r_np).pin_memory(), torch.from_numpy(d_np).pin_memory()
        h_boot = torch.zeros(N, dtype=torch.float32).pin_memory()

        def e2e_rollout(k):
            for t in range(T):
                hts.hts_policy_step_host(ctx, obs_host[(k * T + t) % ring], h_ids, None, t, SEED + k, N,
                                         h_act[t], h_logp[t], h_val[t], h_ent[t], None, s_act)
            hts.hts_gae_host(h_rew, h_val, h_done, h_boot, cfg.gamma, cfg.lam, T, N, h_adv, h_ret, s_act)
        e2e_rollout(0)
        barrier()
        ksteps = max(1, min(args.steps, 3))
        t0 = time.perf_counter()
        for k in range(ksteps):
            e2e_rollout(k + 1)
        torch.cuda.synchronize()
        e2e_s = time.perf_counter() - t0
        if dist is not None:
            ts = torch.tensor([e2e_s], device=dev); dist.all_reduce(ts, op=dist.ReduceOp.MAX); e2e_s = float(ts.item())
        e2e = {"value": world * ksteps * T * N / e2e_s, "unit": UNIT,
               "h2d_bytes_per_step": T * (N * obs_bytes + 4 * N) + 9 * T * N + 4 * N,
               "d2h_bytes_per_step": T * N * 16 + 8 * T * N, "steps": ksteps}
    hts.hts_policy_destroy(ctx)

    # ---- the same actor step at the largest batch of the configurations (cfg5: the whole 8192-env pool,
    #      4x84x84 frames, 18 actions): how the kernels behave when launch and pipeline-fill costs amortise
    big = None
    if rank == 0:
        c5 = wl.CONFIGS[5]
        nb = c5.N
        ctx5 = hts.hts_policy_create(c5.C, c5.H, c5.W, c5.A, hts.HTS_DTYPE_BF16, nb)
        hts.hts_policy_load_weights(ctx5, hts.weights_to_device(wl.make_weights(c5), hts.HTS_DTYPE_BF16, dev))
        obs5 = [torch.from_numpy(wl.make_obs(c5, nb, batch_index=i)).to(dev) for i in range(2)]   # 2 x 231 MB > L2
        ids5 = torch.arange(nb, dtype=torch.int32, device=dev)
        o5 = [torch.empty(nb, dtype=torch.int32, device=dev)] + [torch.empty(nb, device=dev) for _ in range(3)]
        for t in range(5):
            hts.hts_policy_step(ctx5, obs5[t % 2], ids5, None, t, SEED, nb, *o5, None, h_act_stream)
        a5, b5 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        reps = 40
        a5.record(s_act)
        for t in range(reps):
            hts.hts_policy_step(ctx5, obs5[t % 2], ids5, None, t, SEED, nb, *o5, None, h_act_stream)
        b5.record(s_act); torch.cuda.synchronize()
        us5 = 1e3 * a5.elapsed_time(b5) / reps
        tf5 = 2.0 * macs_per_env_step(c5) * nb / (us5 * 1e-6) / 1e12
        hts.hts_policy_profile(ctx5, True)                       # per-kernel event times at this batch
        for t in range(10):
            hts.hts_policy_step(ctx5, obs5[t % 2], ids5, None, t, SEED, nb, *o5, None, h_act_stream)
        torch.cuda.synchronize()
        hts.hts_policy_profile(ctx5, False)
        kern5 = {}
        for i in range(5):
            tot, cnt = hts.hts_policy_profile_read(ctx5, i)
            kern5[hts.hts_policy_kernel_name(i)] = 1e3 * tot / max(cnt, 1)
        big = {"workload": c5.name, "n": nb, "us_per_step": us5, "env_steps_per_s": nb / (us5 * 1e-6), "tflops": tf5,
               "frac_of_bf16_sustained": tf5 / peak_tf, "frac_of_bf16_burst": tf5 / peaks["bf16_tflops"],
               "kernel_us": kern5}
        # the same pool served as the asynchronous executors would hand it over: a random permutation cut into
        # batches of random size 1..4096, each gathered from the state buffer and scattered into the storage row
        batches = [torch.from_numpy(b).to(dev) for b in wl.make_async_batches(c5, nb, 4096)]
        def serve(t):
            for b in batches:
                hts.hts_policy_step_indexed(ctx5, obs5[t % 2], nb, b, b, None, t, SEED, b.numel(), *o5, h_act_stream)
        serve(0)
        a5.record(s_act)
        for t in range(10):
            serve(t)
        b5.record(s_act); torch.cuda.synchronize()
        us_async = 1e3 * a5.elapsed_time(b5) / 10
        big["async_batches"] = {"batches": len(batches), "sizes": [int(b.numel()) for b in batches],
                                "us_per_pool_step": us_async, "env_steps_per_s": nb / (us_async * 1e-6)}
        hts.hts_policy_destroy(ctx5)
        del obs5

    other_configs = config_points(hts, torch, dev, peaks, s_act, l2) if rank == 0 else None

    # ---- the learner's gradient (forward + backward on the fp32 path, CUDA cores, untuned) on one actor batch
    grad_pt = None
    if rank == 0:
        ctxg = hts.hts_policy_create(cfg.C, cfg.H, cfg.W, A, hts.HTS_DTYPE_FP32, N)
        hts.hts_policy_load_weights(ctxg, hts.weights_to_device(params, hts.HTS_DTYPE_FP32, dev))
        grads = {k: torch.empty(v.shape, dtype=torch.float32, device=dev) for k, v in params.items()}
        ga = torch.randint(0, A, (N,), dtype=torch.int32, device=dev)
        gadv, gret = torch.randn(N, device=dev), torch.randn(N, device=dev)
        g_ms = []
        for i in range(5):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(s_act)
            hts.hts_policy_gradient(ctxg, obs_dev[i % ring], ga, gadv, gret, None, 0.5, 0.01, 0.0, N, grads, s_act)
            b.record(s_act); torch.cuda.synchronize()
            g_ms.append(a.elapsed_time(b))
        hts.hts_policy_destroy(ctxg)
        gms = float(np.median(g_ms[1:]))
        gflop = 3 * 2.0 * macs_per_env_step(cfg) * N / 1e9          # forward + data gradient + weight gradient
        grad_pt = {"n": N, "ms": gms, "samples_per_s": N / (gms * 1e-3), "tflops_fp32": gflop / gms,
                   "arithmetic": "fp32 CUDA cores, fixed-order sums", "flops_counted": "3 x forward"}
        del grads

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    # ---- the oracle on this host's cores, bounded sample
    cpu = None
    if not args.no_cpu_baseline:
        from oracle import hts_oracle as orc
        wt = orc.Weights(params)
        rows, nsteps = 1024, 8
        ids = np.arange(rows, dtype=np.int32)
        t0 = time.perf_counter()
        for i in range(nsteps):
            orc.policy_step(wt, obs_host[i % ring].numpy()[:rows], ids, i, SEED)
        ta = time.perf_counter() - t0
        rr, vv, dd, bb = wl.make_rollout(cfg)
        t0 = time.perf_counter()
        orc.gae(rr, vv, dd, bb, cfg.gamma, cfg.lam)
        tg = time.perf_counter() - t0
        cpu = {"value": 1.0 / (ta / (rows * nsteps) + tg / (T * N)), "unit": UNIT, "cores": orc.num_threads(),
               "kind": "oracle",
               "sample": f"{nsteps} actor steps x {rows} envs ({ta:.1f} s) + one full GAE [{T},{N}] ({tg*1e3:.1f} ms)"}

    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": DTYPE, "data": "synthetic",
        "config": {"workload": cfg.name, "N": N, "T": T, "obs": [cfg.C, cfg.H, cfg.W], "actions": A},
        "notes": {"envs_per_gpu": N, "l2": f"observation ring of {ring} batches ({ring * N * obs_bytes >> 20} MiB) exceeds L2 "
                  f"({l2 >> 20} MiB); advantage-scan-alone timings flush L2 between launches",
                  "kernel_times": "second pass over the same rollouts with CUDA events around each kernel"},
        "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches),
        "roofline": roofline,
        "whole_step_tflops": whole_tf, "whole_step_frac_of_bf16_sustained": whole_tf / peak_tf,
        "whole_step_frac_of_bf16_burst": whole_tf / peak_burst,
        "host_enqueue_us_per_actor_step": host_enqueue_us, "overlap": overlap, "configs": other_configs,
        "kernels": kern,
        "gae": {"us_cold": gae_us, "elems_per_s": T * N / (gae_us * 1e-6), "gbs_cold": gae_bytes / (gae_us * 1e-6) / 1e9,
                "wide": {"T": T, "N": Nw, "ms": wide_ms, "gbs": wide_gbs, "elems_per_s": T * Nw / (wide_ms * 1e-3),
                         "frac_of_hbm": wide_gbs / peaks["hbm_gbs"], "peak_gbs": peaks["hbm_gbs"], "peak_kind": peak_kind}},
        "vtrace": {"wide": {"T": T, "N": Nw, "ms": vtrace_ms, "gbs": vtrace_gbs, "elems_per_s": T * Nw / (vtrace_ms * 1e-3),
                            "frac_of_hbm": vtrace_gbs / peaks["hbm_gbs"], "bytes_per_elem": 21}},
        "learner_terms": {"us_cold": terms_us, "elems": T * N,
                          "wide": {"elems": T * Nw, "ms": terms_wide_ms, "gbs": terms_wide_gbs,
                                   "frac_of_hbm": terms_wide_gbs / peaks["hbm_gbs"]},
                          "ppo_wide": {"elems": T * Nw, "ms": ppo_wide_ms, "gbs": ppo_wide_gbs,
                                       "frac_of_hbm": ppo_wide_gbs / peaks["hbm_gbs"],
                                       "bytes_per_elem": "24 (six arrays) + 2 x 4 (advantage mean and variance passes)"}},
        "learner_gradient": grad_pt,
        "delayed_update": {"elems": T * Nw, "ms": upd_wide_ms, "gbs": upd_gbs, "frac_of_hbm": upd_gbs / peaks["hbm_gbs"]},
        "actor_step_us": 1e3 * ms / (args.steps * T),
        "indexed_actor_step_us": indexed_us,
        "large_batch_actor_step": big,
        "cpu_baseline": cpu,
    }
    print(json.dumps(out))
    if dist is not None:
        dist.destroy_process_group()


def rank_env_range(rank: int, envs_per_rank: int) -> tuple[int, int]:
    """Global environment ids of a rank: every rank runs the same per-rank workload on its own id range."""
    return rank * envs_per_rank, (rank + 1) * envs_per_rank


def spawn_command(gpus: int, argv: list[str], port: int | None = None) -> list[str]:
    port = port or int(os.environ.get("MASTER_PORT", "29541"))
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={gpus}",
            "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + list(argv)


def spawn_ranks(gpus: int, argv: list[str]) -> int:
    env = dict(os.environ)
    env.setdefault("NCCL_DEBUG", "INFO")             # the rank count and the transport show up in the log
    return subprocess.call(spawn_command(gpus, argv), env=env)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--ncu-case", type=int, default=0, metavar="STEPS",
                    help="profiling driver: run STEPS actor steps of the bench workload plus one GAE and exit "
                         "(no timing; for use under ncu)")
    ap.add_argument("--ncu-rows", type=int, default=0, metavar="N",
                    help="with --ncu-case: rows per actor step (default: the workload's N)")
    ap.add_argument("--batch-sweep", action="store_true",
                    help="print actor-step time against the batch size (1..8192) and exit")
    ap.add_argument("--ncu-learner-case", action="store_true",
                    help="profiling driver: the HBM-bound kernels (advantage scan, sample means, update) on 2^25 "
                         "transitions, twice each, and exit")
    ap.add_argument("--dry-run-ranks", action="store_true",
                    help="start the ranks as for a real run, print each rank's environment-id range and exit (no GPU work)")
    args = ap.parse_args()
    if args.dry_run_ranks:
        if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
            sys.exit(spawn_ranks(args.gpus, sys.argv[1:]))
        rank, world = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))
        lo, hi = rank_env_range(rank, wl.CONFIGS[WORKLOAD].N)
        print(json.dumps({"rank": rank, "world": world, "env_lo": lo, "env_hi": hi}), flush=True)
        return
    if args.batch_sweep:
        run_batch_sweep()
    elif args.ncu_learner_case:
        run_ncu_learner_case()
    elif args.ncu_case > 0:
        run_ncu_case(args.ncu_case, args.ncu_rows)
    elif args.impl == "reference":
        run_reference(args)
    else:
        if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
            # started without a launcher: start one rank per GPU ourselves (same command line, under torchrun)
            sys.exit(spawn_ranks(args.gpus, sys.argv[1:]))
        run_ours(args)


if __name__ == "__main__":
    main()
