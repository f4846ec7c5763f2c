"""TrainPPO (Algorithm 2) as a sequence of C-ABI calls: GAE once, then for every epoch and
minibatch gather -> forward -> loss -> backward -> Adam, in micro-batches.

Call sequencing and buffer ownership only; all arithmetic happens in libppo_b200.so.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, Optional

import torch

from . import binding as ppo
from .synth import Workload


@dataclass
class Hyper:
    gamma: float = 0.99
    lam: float = 0.95
    clip: float = 0.2
    vf_coef: float = 0.5
    ent_coef: float = 0.01
    lr: float = 3e-4
    beta1: float = 0.9
    beta2: float = 0.999
    eps: float = 1e-8


class Learner:
    def __init__(self, w: Workload, microbatch: int, device="cuda", hyper: Optional[Hyper] = None,
                 with_index: bool = False):
        self.w = w
        self.device = device
        self.hyper = hyper or Hyper(gamma=w.gamma, lam=w.lam, clip=w.clip)
        self.bdesc = ppo.buffer_desc(w.N, w.T, w.H, w.W, w.P, w.A)
        self.buffer = ppo.Buffer(self.bdesc, device)
        self.mdesc = ppo.model_desc(w.H, w.W, w.conv_c, w.conv_k, w.fc, w.P, w.A, norm=w.norm, embed=w.embed,
                                    n_lstm=w.n_lstm, lstm_h=w.lstm_h)
        self.microbatch = min(microbatch, w.B)
        self.recurrent = w.n_lstm > 0
        if self.recurrent:
            # a minibatch is N / minibatches whole env sequences; a micro-batch is a group of them, time-major
            envs = w.N // w.minibatches
            if w.N % w.minibatches:
                raise ValueError("a recurrent minibatch holds whole env sequences: N must divide by minibatches")
            self.seq_envs = max(1, min(self.microbatch // w.T, envs))
            while envs % self.seq_envs:
                self.seq_envs -= 1
            self.microbatch = self.seq_envs * w.T
        self.model = ppo.Model(self.mdesc, self.microbatch, device)
        self.mb = ppo.MinibatchArrays(self.bdesc, self.microbatch if self.recurrent else w.B, device,
                                      with_index=with_index)
        if self.recurrent:
            self.seq_done = torch.zeros((w.T, self.seq_envs), dtype=torch.uint8, device=device)
            self.h_init = torch.zeros((w.n_lstm, self.seq_envs, w.lstm_h), dtype=torch.float32, device=device)
            self.c_init = torch.zeros_like(self.h_init)
        self.roll_h = self.roll_c = self.roll_done = None
        mbs = self.microbatch
        self.mean = torch.empty((mbs, w.A), dtype=torch.float32, device=device)
        self.value = torch.empty(mbs, dtype=torch.float32, device=device)
        self.dmean = torch.empty((mbs, w.A), dtype=torch.float32, device=device)
        self.dvalue = torch.empty(mbs, dtype=torch.float32, device=device)
        self.loss = torch.zeros(5, dtype=torch.float32, device=device)
        self.stats = torch.zeros(2, dtype=torch.float32, device=device)
        self.adam_t = 0

    # ------------------------------------------------------------------ buffer fill

    def write_rollout(self, r: Dict[str, torch.Tensor], action: torch.Tensor, logp: torch.Tensor):
        """D <- D U {...} for t = 0..T-1 from device tensors shaped [T, N, ...]."""
        for t in range(self.w.T):
            ppo.ppo_buffer_write_step(self.buffer, t, r["depth"][t], r["proprio"][t], action[t], logp[t],
                                      r["value"][t], r["reward"][t], r["done"][t])

    def act(self, depth: torch.Tensor, proprio: torch.Tensor, eps: torch.Tensor):
        """Rollout-time policy: mean/value from the encoder, action = mean + sigma * eps and its log-prob.
        depth [n,H,W] fp16, proprio [n,P], eps [n,A]; processed in micro-batches.  Returns (action, logp, value)."""
        n = depth.shape[0]
        action = torch.empty((n, self.w.A), dtype=torch.float32, device=self.device)
        logp = torch.empty(n, dtype=torch.float32, device=self.device)
        value = torch.empty(n, dtype=torch.float32, device=self.device)
        obs = ppo.Minibatch(depth.data_ptr(), proprio.data_ptr(), None, None, None, None, None, None, n)
        if self.recurrent and (self.roll_h is None or self.roll_h.shape[1] != n):
            self.reset_rollout_state(n)
        for r0 in range(0, n, self.microbatch):
            rows = min(self.microbatch, n - r0)
            if self.recurrent:  # a one-step sequence from the state the envs carry
                h_in = self.roll_h[:, r0:r0 + rows].contiguous()
                c_in = self.roll_c[:, r0:r0 + rows].contiguous()
                ppo.ppo_model_set_sequence(self.model, 1, rows, self.roll_done[r0:r0 + rows], h_in, c_in)
            ppo.ppo_encoder_fwd(self.model, obs, r0, rows, self.mean, value[r0:r0 + rows])
            ppo.ppo_policy_sample(self.model, rows, self.mean, eps[r0:r0 + rows], action[r0:r0 + rows],
                                  logp[r0:r0 + rows])
            if self.recurrent:  # the state these envs carry into their next step
                ppo.ppo_model_read_state(self.model, h_in, c_in)
                self.roll_h[:, r0:r0 + rows] = h_in
                self.roll_c[:, r0:r0 + rows] = c_in
        return action, logp, value

    def reset_rollout_state(self, n: int, done: Optional[torch.Tensor] = None):
        """Recurrent state the rollout policy carries per env: all zeros (done None), or zeroed where done != 0."""
        w = self.w
        if done is None or self.roll_h is None:
            self.roll_h = torch.zeros((w.n_lstm, n, w.lstm_h), dtype=torch.float32, device=self.device)
            self.roll_c = torch.zeros_like(self.roll_h)
            self.roll_done = torch.zeros(n, dtype=torch.uint8, device=self.device)
        else:
            keep = (done == 0).to(torch.float32).view(1, n, 1)
            self.roll_h *= keep
            self.roll_c *= keep

    def act_into_buffer(self, t: int, depth: torch.Tensor, proprio: torch.Tensor, eps: torch.Tensor):
        """One rollout step without intermediate copies: the observation goes into slab row t, the policy reads
        it there and writes action, log-prob and value into the same row (Algorithm 2, actions <- pi(obs) then
        D <- D U {...}); ppo_buffer_write_outcome adds reward and done once the env has stepped."""
        if self.recurrent:
            raise NotImplementedError("a recurrent policy acts through act(), which carries the state")
        ppo.ppo_buffer_write_obs(self.buffer, t, depth, proprio)
        ppo.ppo_policy_act(self.model, self.buffer, t, eps)

    # ------------------------------------------------------------------ TrainPPO

    def compute_gae(self, last_value: torch.Tensor, normalize: bool = True):
        h = self.hyper
        ppo.ppo_compute_gae(self.buffer, last_value, h.gamma, h.lam, normalize, self.stats)

    def minibatch_step(self, seed: int, epoch: int, k: int, num_minibatches: Optional[int] = None):
        """gather -> (fwd -> loss -> bwd) per micro-batch -> Adam for minibatch k of this epoch."""
        w, h = self.w, self.hyper
        K = num_minibatches or w.minibatches
        B = w.M // K
        if self.recurrent:
            return self._sequence_step(seed, epoch, k, K)
        ppo.ppo_shuffle_gather_minibatch(self.buffer, seed, epoch, k, K, self.mb)
        ppo.ppo_model_zero_grad(self.model)
        self.loss.zero_()
        for r0 in range(0, B, self.microbatch):
            rows = min(self.microbatch, B - r0)
            ppo.ppo_encoder_fwd(self.model, self.mb, r0, rows, self.mean, self.value)
            ppo.ppo_loss_fwd_bwd(self.model, self.mb, r0, rows, B, self.mean, self.value, h.clip, h.vf_coef,
                                 h.ent_coef, self.loss, self.dmean, self.dvalue)
            ppo.ppo_encoder_bwd(self.model, self.mb, r0, rows, self.dmean, self.dvalue, True)
        self.adam_t += 1
        ppo.ppo_adam_step(self.model, h.lr, h.beta1, h.beta2, h.eps, self.adam_t)

    def _sequence_step(self, seed: int, epoch: int, k: int, K: int):
        """Recurrent minibatch k: the env permutation is cut into K * S groups of seq_envs envs, groups k*S .. k*S+S-1
        are this minibatch's micro-batches; each runs forward through time from a zero state (reset again wherever
        the previous step ended an episode), then backward through time."""
        w, h = self.w, self.hyper
        S = (w.N // K) // self.seq_envs
        rows, B = self.microbatch, (w.N // K) * w.T
        ppo.ppo_model_zero_grad(self.model)
        self.loss.zero_()
        for j in range(S):
            ppo.ppo_shuffle_gather_sequences(self.buffer, seed, epoch, k * S + j, K * S, self.mb, self.seq_done)
            ppo.ppo_model_set_sequence(self.model, w.T, self.seq_envs, self.seq_done, self.h_init, self.c_init)
            ppo.ppo_encoder_fwd(self.model, self.mb, 0, rows, self.mean, self.value)
            ppo.ppo_loss_fwd_bwd(self.model, self.mb, 0, rows, B, self.mean, self.value, h.clip, h.vf_coef,
                                 h.ent_coef, self.loss, self.dmean, self.dvalue)
            ppo.ppo_encoder_bwd(self.model, self.mb, 0, rows, self.dmean, self.dvalue, True)
        self.adam_t += 1
        ppo.ppo_adam_step(self.model, h.lr, h.beta1, h.beta2, h.eps, self.adam_t)

    def train(self, last_value: torch.Tensor, seed: int = 0):
        """One TrainPPO call over the current buffer."""
        self.compute_gae(last_value)
        for e in range(self.w.epochs):
            for k in range(self.w.minibatches):
                self.minibatch_step(seed, e, k)
