"""Convenience driver of one full pass (build tree -> reward -> surrogate gradient).

Owns a library context and the caller-side buffers; every step is one C-ABI call.
"""
from __future__ import annotations

import numpy as np
import torch

from . import binding as gto
from . import synth


class GtoPass:
    def __init__(self, w: synth.Workload, device="cuda:0", reward_agg=gto.GTO_AGG_LSE, flags=0):
        self.w = w
        self.device = torch.device(device)
        idx = self.device.index if self.device.index is not None else torch.cuda.current_device()
        self.cfg = gto.make_config(w.B, w.D, w.k, w.g, w.m, w.V_draft, w.V_target, w.dtype, G=w.G,
                                   eta=w.eta, clip_eps=w.clip_eps, std_delta=w.std_delta,
                                   grad_scale=w.grad_scale, reward_agg=reward_agg, flags=flags)
        self.ctx = gto.gto_create(self.cfg, idx)
        self.tree = gto.alloc_tree(self.cfg, self.device)
        self.reward = gto.alloc_reward(self.cfg, self.device)
        self.stats = gto.alloc_grad_stats(self.cfg, self.device)
        self.grad = torch.empty((w.B, w.D, w.V_draft), dtype=w.torch_dtype, device=self.device)
        self.old_logp = torch.zeros((w.B, w.D), dtype=torch.float32, device=self.device)

    def close(self):
        if self.ctx is not None:
            gto.gto_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- the three entry points
    def build_tree(self, draft, stream=None):
        gto.gto_build_tree(self.ctx, draft, self.tree, stream)

    def tree_reward(self, target, d2t, stream=None):
        gto.gto_tree_reward(self.ctx, self.tree, target, d2t, self.reward, stream)

    def tree_reward_host(self, target_host, target_dev, d2t, stream=None) -> int:
        return gto.gto_tree_reward_host(self.ctx, self.tree, target_host, target_dev, d2t, self.reward,
                                        stream)

    def surrogate_grad(self, draft, stream=None):
        gto.gto_group_surrogate_grad(self.ctx, draft, self.tree, self.reward, self.old_logp,
                                     self.grad, self.stats, stream)

    def set_old_logp_from_path(self, b0: int = 0):
        """Old-policy log-probabilities of the accepted paths (an input of the gradient
        call): the reported path log-probabilities plus the seeded perturbation."""
        r = self.reward
        old = synth.old_logp_from_path(self.w, r["path_logp"].cpu().numpy().astype(np.float64),
                                       r["path_row"].cpu().numpy(), r["path_token"].cpu().numpy(),
                                       r["path_len"].cpu().numpy(), b0=b0)
        self.old_logp.copy_(torch.from_numpy(old).to(torch.float32))

    def step(self, draft, target, d2t, stream=None):
        """One pass with the current old_logp buffer."""
        self.build_tree(draft, stream)
        self.tree_reward(target, d2t, stream)
        self.surrogate_grad(draft, stream)

    def token_loss(self, draft, target, d2t, weight: float = 1.0, stream=None):
        """Token-level loss on the root rows; allocates its outputs on first use."""
        if not hasattr(self, "token_stats"):
            self.token_stats = gto.alloc_token_stats(self.cfg, self.device)
            self.grad_root = torch.empty((self.w.B, self.w.V_draft), dtype=self.w.torch_dtype,
                                         device=self.device)
        gto.gto_token_loss(self.ctx, draft, target, d2t, self.tree, weight, self.grad_root,
                           self.token_stats, stream)

    def token_loss_accumulate(self, draft, target, d2t, weight: float = 1.0, stream=None):
        """Token-level loss added into slice [b, 0, :] of the surrogate gradient buffer."""
        if not hasattr(self, "token_stats"):
            self.token_stats = gto.alloc_token_stats(self.cfg, self.device)
        gto.gto_token_loss_accumulate(self.ctx, draft, target, d2t, self.tree, self.reward, self.stats,
                                      weight, self.grad, self.token_stats, stream)

    def status(self) -> int:
        return gto.gto_device_status(self.ctx)

    def launches(self) -> int:
        return gto.gto_launch_count(self.ctx)
