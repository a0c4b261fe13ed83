"""Sequences the C-ABI calls of one batch of rollout trees for a workload.

PyTorch is used for device memory, host<->device copies and streams only; every
step of the method is a call into libbgrpo.so through ``binding``.
"""
from __future__ import annotations

import math
from typing import Optional

import numpy as np
import torch

from . import binding as B


class TreeSession:
    """Device buffers + handle for `n_trees` trees of one workload shape.

    Order of calls (Algorithm 1 of the paper, per prompt): rollout() = tree_init, then T x
    [velocity, tree_step]; rewards(); fuse_advantage(); prune().
    """

    def __init__(self, w, n_trees: Optional[int] = None, tree_id_base: int = 0, device="cuda:0", nodes_cap=None,
                 fused_rollout: bool = False):
        self.w = w
        # one launch for all T steps (closed-form velocity only) instead of one tree_step per depth
        self.fused_rollout = fused_rollout and w.velocity == "linear"
        self.n_trees = w.n_trees if n_trees is None else n_trees
        self.device = torch.device(device)
        self.nodes_cap = w.nodes if nodes_cap is None else nodes_cap
        self.desc, self._grid = B.make_desc(self.n_trees, w.tokens, w.channels, w.T, w.K, self.nodes_cap,
                                           float(np.float32(w.sigma)), w.t_grid(), w.seed,
                                           branch_corr_s=w.branch_corr_s, tree_id_base=tree_id_base)
        sz = B.tree_workspace(self.desc)
        rows = self.n_trees * self.nodes_cap
        dev = self.device
        self.latents = torch.empty(sz.latents_bytes // 4, dtype=torch.float32, device=dev).view(self.n_trees, self.nodes_cap, w.D)
        self.node_table = torch.empty((4, rows), dtype=torch.int32, device=dev)
        self.logp = torch.empty((self.n_trees, self.nodes_cap), dtype=torch.float32, device=dev)
        self.rbar = torch.empty_like(self.logp)
        self.adv = torch.empty_like(self.logp)
        self.mask = torch.empty((self.n_trees, self.nodes_cap), dtype=torch.uint8, device=dev)
        self.scratch = torch.empty(sz.scratch_bytes, dtype=torch.uint8, device=dev)
        self.leaf_r = torch.empty((self.n_trees, w.leaves), dtype=torch.float32, device=dev)
        self.tree = None
        self.mu = self.target = self.packed = self.v = self.reward_draws = None
        self.pruned_steps = ()
        self._split_flags = np.ascontiguousarray([1 if i in w.splits else 0 for i in range(w.T)], dtype=np.uint8)

    # -- inputs ---------------------------------------------------------------------------------------------------
    def upload_inputs(self, inp):
        """Copies the seeded inputs of `workloads.make_inputs` to the device."""
        dev = self.device
        w = self.w
        if inp.mu is not None:
            self.mu = torch.from_numpy(inp.mu).to(dev)
        if inp.target is not None:
            self.target = torch.from_numpy(inp.target).to(dev)
        if inp.reward_draws is not None:
            self.reward_draws = torch.from_numpy(inp.reward_draws).to(dev)
        if inp.W1 is not None:
            from workloads import bf16_bits
            W1 = torch.from_numpy(bf16_bits(inp.W1).view(np.int16)).to(dev)
            W2 = torch.from_numpy(bf16_bits(inp.W2).view(np.int16)).to(dev)
            nbytes = B.velocity_mlp_packed_bytes(w.hidden)
            self.packed = torch.empty(nbytes + 1024, dtype=torch.uint8, device=dev)
            off = (-self.packed.data_ptr()) % 1024
            self.packed = self.packed[off:off + nbytes]
            B.velocity_mlp_pack(W1, W2, w.hidden, self.packed)
            torch.cuda.synchronize()
            self.v = torch.empty((self.n_trees, w.leaves, w.D), dtype=torch.float32, device=dev)
        self.pruned_steps = tuple(int(x) for x in inp.pruned_steps)

    # -- the path -------------------------------------------------------------------------------------------------
    def init(self, seed=None):
        if self.tree is None:
            if seed is not None:
                self.desc.seed = seed
            self.tree = B.tree_init(self.desc, self.latents, self.node_table, self.logp, self.rbar, self.adv, self.mask,
                                    self.scratch, keep=(self._grid,))
            if self.mu is not None:
                B.velocity_linear_bind(self.tree, self.mu, float(np.float32(self.w.s0)))
        else:
            B.tree_reset(self.tree, self.desc.seed if seed is None else seed)

    def step(self, i: int, v=None):
        split = 1 if i in self.w.splits else 0
        if v is None and self.w.velocity == "mlp":
            B.velocity_mlp(self.tree, self.packed, self.w.hidden, self.v)
            v = self.v
        B.tree_step(self.tree, split, v)

    def rollout(self, seed=None):
        self.init(seed)
        if self.fused_rollout:
            B.tree_rollout_fused(self.tree, self._split_flags)
        elif self.w.velocity == "mlp":
            B.tree_rollout(self.tree, self._split_flags, self.packed, self.w.hidden, self.v)       # T x [velocity, step], one host call
        else:
            B.tree_rollout(self.tree, self._split_flags)

    def rewards(self):
        w = self.w
        if w.reward == "neg_mse_mu":
            B.leaf_reward_mse(self.tree, self.mu, self.leaf_r)
        elif w.reward == "neg_mse_target":
            B.leaf_reward_mse(self.tree, self.target, self.leaf_r)
        elif w.reward == "normal_plus_cos":
            self.leaf_r.copy_(self.reward_draws)
            B.leaf_reward_cos(self.tree, self.target, 0.1, self.leaf_r)
        elif w.reward == "mixture":
            self.leaf_r.copy_(self.reward_draws)
        else:
            raise ValueError(w.reward)

    def fuse_advantage(self):
        w = self.w
        B.tree_fuse_advantage(self.tree, self.leaf_r, float(np.float32(w.beta)), 1.0, float(np.float32(w.eps)),
                              float(np.float32(w.adv_clip)))

    def prune(self):
        w = self.w
        B.tree_prune(self.tree, w.width_mode, w.width_k, self.pruned_steps, w.ignore_last_step)

    def run_all(self, seed=None):
        """One pass of the whole path over this batch."""
        self.rollout(seed)
        self.rewards()
        self.fuse_advantage()
        self.prune()

    def kernel_launches_per_pass(self) -> int:
        w = self.w
        if self.fused_rollout:
            n = 1 + 2                                              # root + whole-tree rollout + its log-prob sums
        else:
            n = 1 + w.T * (2 if w.velocity == "mlp" else 1) + 1   # root + (mlp +) step per depth + log-prob flush
        n += 2 if w.reward in ("neg_mse_mu", "neg_mse_target", "normal_plus_cos") else 0   # partial sums + their fixed-order total
        n += 2                                                     # fuse+advantage, prune
        return n
