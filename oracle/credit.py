"""Credit assignment on a rollout tree (oracle, test infrastructure): reward fusion
(Eq. 3), depth-wise normalisation (Eq. 4) and the pruning masks of the "Pruning
Strategies" section.  All arithmetic is float64.

Readings where the paper is silent
----------------------------------
* N_d of Eq. 4 is the set of depth-d nodes of ONE prompt's tree; sigma_d is the
  population standard deviation, so a depth with a single node gets A = 0.
* The root has no incoming edge: its advantage is 0 and its mask is 0.
* Width pruning has three modes: top-k children at every split (the ablation's
  reading of Parent-Top1), top-k children at the last split only (the method
  section's reading, "Width Pruning") and Extreme-b (best b and worst b leaves).
  A pruned child loses
  its incoming edge and its whole subtree; ancestors it shares with kept
  children stay.  Ties rank the lower branch index (or leaf index) first.
* Depth pruning is indexed by step: step i in the pruned set removes the edges
  i -> i+1, i.e. the nodes of depth i+1.
* The sliding window of the ablation "Pruning Strategies" (it starts at the last
  split step, spans four steps and moves one step deeper every thirty iterations,
  up to a stop depth) gives steps min(start + iter // every, stop - size) + 0..size-1.
"""
from __future__ import annotations

import math
from typing import Iterable, Optional, Sequence

import numpy as np

from .tree import Topology

WIDTH_NONE = 0
WIDTH_PER_SPLIT_TOPK = 1
WIDTH_LAST_SPLIT_TOPK = 2
WIDTH_EXTREME_B = 3


def path_logp(topo: Topology, edge_logp: np.ndarray, n: int, leaf: int) -> float:
    """s_l = log p_beh(l | n): sum of the edge log-probs on the path from n down to leaf l."""
    s, m = 0.0, leaf
    while m != n:
        s += float(edge_logp[m])
        m = int(topo.parent[m])
        assert m >= 0, "leaf is not a descendant of n"
    return s


def fuse_rewards(topo: Topology, leaf_rewards: Sequence[float], edge_logp: Optional[np.ndarray] = None,
                 beta: float = 0.0, logp_scale: float = 1.0) -> np.ndarray:
    """rbar(n) = sum_{l in L(n)} softmax_l(beta * s_l) r_l  for every node (Eq. 3), by direct
    enumeration of each node's descendant leaves.  edge_logp[c] is the log-prob of the edge
    into node c (times logp_scale, e.g. D to turn a per-element mean into a joint log-density)."""
    r = np.asarray(leaf_rewards, dtype=np.float64)
    assert r.shape == (topo.leaves,)
    first_leaf = topo.offset[topo.T]
    rbar = np.zeros(topo.nodes, dtype=np.float64)
    for n in range(topo.nodes):
        leaves = topo.descendant_leaves(n)
        if beta == 0.0 or edge_logp is None:
            a = np.zeros(len(leaves))
        else:
            a = np.array([beta * logp_scale * path_logp(topo, edge_logp, n, l) for l in leaves])
        w = np.exp(a - a.max())
        w /= w.sum()
        rbar[n] = float(np.dot(w, r[[l - first_leaf for l in leaves]]))
    return rbar


def fusion_ess(topo: Topology, edge_logp: Optional[np.ndarray] = None, beta: float = 0.0,
               logp_scale: float = 1.0) -> np.ndarray:
    """Effective sample size of the fusion weights of every node (appendix "Reward Fusion: Unbiasedness and
    Variance Reduction"): ESS(n) = (sum_l w_l)^2 / sum_l w_l^2 over the descendant leaves of n, with the
    weights of Eq. 3, w_l proportional to exp(beta * s_l).  By direct enumeration, like fuse_rewards.
    beta = 0 gives |L(n)|; one dominant leaf gives 1."""
    ess = np.zeros(topo.nodes, dtype=np.float64)
    for n in range(topo.nodes):
        leaves = topo.descendant_leaves(n)
        if beta == 0.0 or edge_logp is None:
            a = np.zeros(len(leaves))
        else:
            a = np.array([beta * logp_scale * path_logp(topo, edge_logp, n, l) for l in leaves])
        w = np.exp(a - a.max())
        ess[n] = float(w.sum() ** 2 / (w ** 2).sum())
    return ess


def depth_advantages(topo: Topology, rbar: np.ndarray, eps: float = 1e-6, clip: float = 0.0) -> np.ndarray:
    """A_d(n) = (rbar(n) - mu_d) / (sigma_d + eps) over the nodes of each depth d >= 1 (Eq. 4);
    the edge into n carries A(n); optional clipping to [-clip, clip] when clip > 0."""
    rbar = np.asarray(rbar, dtype=np.float64)
    adv = np.zeros(topo.nodes, dtype=np.float64)
    for d in range(1, topo.T + 1):
        idx = list(topo.level(d))
        x = rbar[idx]
        mu = x.mean()
        sd = math.sqrt(((x - mu) ** 2).mean())
        adv[idx] = (x - mu) / (sd + eps)
    if clip > 0:
        adv = np.clip(adv, -clip, clip)
    return adv


def width_keep(topo: Topology, rbar: np.ndarray, mode: int, k: int) -> np.ndarray:
    """keep_w[n] in {0,1}: whether node n (and the edge into it) survives width pruning."""
    keep = np.ones(topo.nodes, dtype=np.uint8)
    if mode == WIDTH_NONE:
        return keep
    if mode == WIDTH_EXTREME_B:
        leaves = list(topo.leaf_ids())
        vals = [float(rbar[l]) for l in leaves]
        best = sorted(range(len(leaves)), key=lambda q: (-vals[q], q))[:k]
        worst = sorted(range(len(leaves)), key=lambda q: (vals[q], q))[:k]
        keep[:] = 0
        for q in set(best) | set(worst):
            for m in topo.path_to_root(leaves[q]):
                keep[m] = 1
        return keep
    last_split = max(topo.splits) if topo.splits else -1
    for i in range(topo.T):
        ranked_here = (i in topo.splits) and (mode == WIDTH_PER_SPLIT_TOPK or i == last_split)
        for p in topo.level(i):
            kids = topo.children(p)
            order = sorted(range(len(kids)), key=lambda b: (-float(rbar[kids[b]]), b))
            for rank, b in enumerate(order):
                ok = keep[p] and (not ranked_here or rank < k)
                keep[kids[b]] = 1 if ok else 0
    return keep


def depth_keep(topo: Topology, pruned_steps: Iterable[int]) -> np.ndarray:
    """keep_d[n] = 0 for nodes of depth i+1 with step i in the pruned set D."""
    keep = np.ones(topo.nodes, dtype=np.uint8)
    pruned = set(int(i) for i in pruned_steps)
    for n in range(topo.nodes):
        if int(topo.depth[n]) - 1 in pruned:
            keep[n] = 0
    return keep


def gradient_mask(topo: Topology, rbar: np.ndarray, width_mode: int, k: int,
                  pruned_steps: Iterable[int] = (), ignore_last_step: bool = False, sde_steps=None) -> np.ndarray:
    """mask[n] = 1 iff the node-step (edge) into n receives gradients.  With a hybrid ODE-SDE
    schedule (sde_steps given) the deterministic ODE steps have no transition density and are masked."""
    m = width_keep(topo, rbar, width_mode, k) & depth_keep(topo, pruned_steps)
    if sde_steps is not None:
        m &= depth_keep(topo, [i for i in range(topo.T) if i not in set(int(x) for x in sde_steps)])
    m[0] = 0
    if ignore_last_step:   # "Ignore last step: Yes" (hyper-parameter table)
        m[list(topo.level(topo.T))] = 0
    return m


def depth_window(iteration: int, start: int, size: int = 4, every: int = 30, stop: Optional[int] = None):
    """Pruned steps of the sliding window at a training iteration."""
    first = start + iteration // every
    if stop is not None:
        first = min(first, stop - size)
    return [first + j for j in range(size)]


def grpo_objective(topo: Topology, logp_new: np.ndarray, logp_old: np.ndarray, adv: np.ndarray, mask: np.ndarray,
                   clip_eps: float, logp_scale: float = 1.0):
    """Forward value of the clipped GRPO objective over the tree's edges (Eq. 5):
        J = 1/|E| sum_e min(rho_e A(e), clip(rho_e, 1 - eps, 1 + eps) A(e)),   rho_e = pi_new(e) / pi_old(e),
    with E the edges that receive gradients (mask) and rho_e = exp(logp_scale (logp_new - logp_old)).
    Returns (J, per-edge terms with 0 on unmasked nodes).  An empty edge set gives J = 0."""
    terms = np.zeros(topo.nodes, dtype=np.float64)
    n = 0
    for e in range(1, topo.nodes):
        if not mask[e]:
            continue
        rho = math.exp(logp_scale * (float(logp_new[e]) - float(logp_old[e])))
        a = float(adv[e])
        terms[e] = min(rho * a, min(max(rho, 1.0 - clip_eps), 1.0 + clip_eps) * a)
        n += 1
    return (float(terms.sum() / n) if n else 0.0), terms


def mix_sde_steps(T: int, splits: Sequence[int], iteration: int, window: int = 4, every: int = 30, start: int = 0):
    """Hybrid ODE-SDE schedule: every branching step plus a sliding window of `window` further steps (same
    window rule as depth pruning: one step deeper every `every` iterations, kept inside 0..T-1)."""
    first = min(start + iteration // every, max(T - window, 0))
    return sorted(set(int(x) for x in splits) | set(range(first, min(first + window, T))))
