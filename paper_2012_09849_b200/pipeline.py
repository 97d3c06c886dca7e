"""Two-storage rollout schedule: the actor steps of rollout k+1 overlap the advantage scan of rollout k.

Section 4.1 of the paper ("two data storages", "Concurrent rollout and learning"): while the learner
consumes one storage, the actors fill the other, and the two swap roles once per rollout.  Here the
consumer is the advantage scan and the swap is three CUDA events per storage:

    filled    all T actor steps of the storage have been written        (recorded on the actor stream)
    row0      its value row 0 has been written                          (recorded on the actor stream)
    consumed  the scan that reads it has finished                       (recorded on the scan stream)

Rollout k writes storage k % 2 on the actor stream (after `consumed` of that storage); the scan of
rollout k-1 runs on the scan stream after `filled` of its storage and `row0` of rollout k, because its
bootstrap V(s_T) is the value row 0 of rollout k (the states a rollout ends in are the states the next one
starts from).  This module only enqueues: every arithmetic step is a call of the C ABI.
"""
from __future__ import annotations

import torch

from . import (hts_gae, hts_policy_step)


class Storage:
    """One of the two [T, N] rollout storages, with the raw row addresses the timed loop uses."""

    def __init__(self, T: int, N: int, device):
        self.actions = torch.empty(T, N, dtype=torch.int32, device=device)
        self.logp = torch.empty(T, N, dtype=torch.float32, device=device)
        self.values = torch.empty(T, N, dtype=torch.float32, device=device)
        self.entropy = torch.empty(T, N, dtype=torch.float32, device=device)
        self.adv = torch.empty(T, N, dtype=torch.float32, device=device)
        self.ret = torch.empty(T, N, dtype=torch.float32, device=device)
        self.filled = torch.cuda.Event()
        self.row0 = torch.cuda.Event()
        self.consumed = torch.cuda.Event()
        self.p_act = [self.actions[t].data_ptr() for t in range(T)]
        self.p_logp = [self.logp[t].data_ptr() for t in range(T)]
        self.p_val = [self.values[t].data_ptr() for t in range(T)]
        self.p_ent = [self.entropy[t].data_ptr() for t in range(T)]


class RolloutPipeline:
    """Enqueues rollouts of T actor steps over N environments on one stream and the advantage scan of
    the previous rollout on a second one.

    obs_for(k, t) -> address (or tensor) of the uint8 [N,C,H,W] frames of step t of rollout k;
    seed_for(k)   -> the 64-bit seed of rollout k;
    rewards, dones: [T, N] device tensors read by every scan (synthetic environments have no feedback
    from the actions, so one pair serves all rollouts); `after_scan(k, storage)`, if given, is called
    right after the scan of rollout k has been enqueued (tests use it to copy results out on the scan
    stream before the storage is reused).
    """

    def __init__(self, ctx, T, N, env_ids, rewards, dones, gamma, lam, obs_for, seed_for, device=None,
                 overlap=True, after_scan=None):
        device = device or env_ids.device
        self.ctx, self.T, self.N = ctx, T, N
        self.env_ids, self.rewards, self.dones = env_ids, rewards, dones
        self.gamma, self.lam = gamma, lam
        self.obs_for, self.seed_for, self.after_scan = obs_for, seed_for, after_scan
        self.store = [Storage(T, N, device), Storage(T, N, device)]
        self.s_act = torch.cuda.Stream(device)
        # the scan runs at high priority: its blocks take the SMs that the persistent actor kernels free at their
        # tails instead of queueing behind the next actor kernel
        self.s_gae = torch.cuda.Stream(device, priority=-1) if overlap else self.s_act
        for s in self.store:
            s.consumed.record(self.s_gae); s.filled.record(self.s_act); s.row0.record(self.s_act)
        self._p_ids = env_ids.data_ptr()
        self._h_act, self._h_gae = self.s_act.cuda_stream, self.s_gae.cuda_stream
        self.started = False

    def rollout(self, k: int) -> None:
        """Actor steps of rollout k, then (if a previous rollout exists) the scan of rollout k-1."""
        cur, prev = self.store[k % 2], self.store[(k + 1) % 2]
        T, N = self.T, self.N
        self.s_act.wait_event(cur.consumed)                          # the storage is free again (role swap)
        seed = self.seed_for(k)
        for t in range(T):
            hts_policy_step(self.ctx, self.obs_for(k, t), self._p_ids, None, t, seed, N,
                            cur.p_act[t], cur.p_logp[t], cur.p_val[t], cur.p_ent[t], None, self._h_act)
            if t == 0:
                cur.row0.record(self.s_act)
        cur.filled.record(self.s_act)
        if self.started:
            self.s_gae.wait_event(prev.filled)
            self.s_gae.wait_event(cur.row0)
            hts_gae(self.rewards, prev.values, self.dones, cur.p_val[0], self.gamma, self.lam, T, N,
                    prev.adv, prev.ret, self._h_gae)
            if self.after_scan is not None:
                self.after_scan(k - 1, prev)
            prev.consumed.record(self.s_gae)
        self.started = True

    def join(self) -> None:
        """Make the actor stream wait for the scan stream (so one event on the actor stream closes both)."""
        if self.s_gae is not self.s_act:
            self.s_act.wait_stream(self.s_gae)
