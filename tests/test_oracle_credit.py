"""Pins for oracle/credit.py: special cases the paper states (beta = 0, beta = 1), library
softmax / z-score, hand-worked tiny trees, brute-force counts of the masks."""
import math

import numpy as np
import pytest
from scipy import special, stats

from oracle import credit, tree


def _random_case(T, K, splits, seed=0):
    topo = tree.build_topology(T, K, splits)
    rng = np.random.default_rng(seed)
    r = rng.standard_normal(topo.leaves)
    logp = -np.abs(rng.standard_normal(topo.nodes))
    logp[0] = 0.0
    return topo, r, logp


def test_beta_zero_is_the_mean_of_descendant_leaves():
    topo, r, logp = _random_case(6, 3, (0, 2, 5))
    rbar = credit.fuse_rewards(topo, r, logp, beta=0.0)
    # independent route: bottom-up (sum, count) accumulation
    tot = np.zeros(topo.nodes)
    cnt = np.zeros(topo.nodes)
    first = topo.offset[topo.T]
    tot[first:] = r
    cnt[first:] = 1
    for n in range(topo.nodes - 1, 0, -1):
        tot[topo.parent[n]] += tot[n]
        cnt[topo.parent[n]] += cnt[n]
    assert np.allclose(rbar, tot / cnt, rtol=1e-13)
    assert math.isclose(rbar[0], r.mean(), rel_tol=1e-13)
    assert np.array_equal(rbar[first:], r)


def test_beta_one_weights_by_behaviour_probability():
    """Hand-worked: root -> 2 children (p = 0.25, 0.75), second child -> 2 leaves (p = 0.1, 0.9)
    after a split; first child's subtree likewise with (0.5, 0.5)."""
    topo = tree.build_topology(2, 2, (0, 1))
    # nodes: 0 | 1 2 | 3 4 5 6 ; leaves 3,4 under 1 and 5,6 under 2
    p = np.array([1.0, 0.25, 0.75, 0.5, 0.5, 0.1, 0.9])
    logp = np.log(p)
    r = np.array([1.0, 3.0, -2.0, 4.0])
    rbar = credit.fuse_rewards(topo, r, logp, beta=1.0)
    assert math.isclose(rbar[1], 0.5 * 1 + 0.5 * 3, rel_tol=1e-14)
    assert math.isclose(rbar[2], 0.1 * -2 + 0.9 * 4, rel_tol=1e-14)
    # at the root p(l | root) = product along the path, already normalised
    w = np.array([0.25 * 0.5, 0.25 * 0.5, 0.75 * 0.1, 0.75 * 0.9])
    assert math.isclose(rbar[0], float(w @ r), rel_tol=1e-14)
    # a shift common to the edges of a depth (unnormalised probabilities) is removed by the softmax
    rbar2 = credit.fuse_rewards(topo, r, logp + np.array([0, -3.0, -3.0, 1.5, 1.5, 1.5, 1.5]), beta=1.0)
    assert np.allclose(rbar2, rbar, rtol=1e-13)


def test_general_beta_equals_library_softmax_and_scale():
    topo, r, logp = _random_case(5, 2, (0, 1, 3), seed=3)
    first = topo.offset[topo.T]
    for beta, scale in ((0.5, 1.0), (2.0, 1.0), (1.0, 7.0)):
        rbar = credit.fuse_rewards(topo, r, logp, beta=beta, logp_scale=scale)
        for n in (0, 1, 2, 5):
            ls = topo.descendant_leaves(n)
            s = np.array([sum(logp[m] for m in topo.path_to_root(l) if topo.depth[m] > topo.depth[n]) for l in ls])
            w = special.softmax(beta * scale * s)
            assert math.isclose(rbar[n], float(w @ r[[l - first for l in ls]]), rel_tol=1e-12)
    # equal edge log-probs make the fusion independent of beta
    flat = np.full(topo.nodes, -1.7)
    assert np.allclose(credit.fuse_rewards(topo, r, flat, beta=3.0), credit.fuse_rewards(topo, r, flat, beta=0.0), rtol=1e-13)
    # huge scales do not overflow (softmax is shift-invariant)
    big = credit.fuse_rewards(topo, r, logp, beta=1.0, logp_scale=1e6)
    assert np.all(np.isfinite(big))
    # single-child chains copy the child's value
    for n in range(topo.nodes):
        kids = topo.children(n)
        if len(kids) == 1:
            assert big[n] == big[kids[0]]


def test_depth_advantages_are_library_zscores():
    topo, r, logp = _random_case(6, 2, (0, 2, 4), seed=5)
    rbar = credit.fuse_rewards(topo, r, logp, beta=1.0)
    adv = credit.depth_advantages(topo, rbar, eps=0.0)
    for d in range(1, topo.T + 1):
        idx = list(topo.level(d))
        if len(idx) > 1:
            assert np.allclose(adv[idx], stats.zscore(rbar[idx], ddof=0), rtol=1e-12, atol=1e-12)
            assert abs(adv[idx].sum()) < 1e-12          # zero mean: sum_b A = 0
            assert math.isclose(np.mean(adv[idx] ** 2), 1.0, rel_tol=1e-12)
    assert adv[0] == 0.0
    # eps shrinks by sigma / (sigma + eps); leaves at beta = 0 give the GRPO group z-score
    eps = 0.25
    adv_e = credit.depth_advantages(topo, rbar, eps=eps)
    idx = list(topo.level(topo.T))
    sd = rbar[idx].std()
    assert np.allclose(adv_e[idx], adv[idx] * sd / (sd + eps), rtol=1e-12)
    leaves0 = credit.depth_advantages(topo, credit.fuse_rewards(topo, r, None, 0.0), eps=0.0)[idx]
    assert np.allclose(leaves0, (r - r.mean()) / r.std(), rtol=1e-12)


def test_single_node_depths_and_clip():
    topo = tree.build_topology(4, 2, (2,))
    r = np.array([10.0, -10.0])
    rbar = credit.fuse_rewards(topo, r, None, 0.0)
    adv = credit.depth_advantages(topo, rbar, eps=1e-6)
    assert np.all(adv[:3] == 0.0)                   # depths 0..2 hold one node each
    assert np.allclose(adv[-2:], [1.0, -1.0], atol=1e-6)
    assert np.array_equal(credit.depth_advantages(topo, rbar, eps=1e-6, clip=0.5)[-2:], [0.5, -0.5])


def _kept_leaves(topo, keep):
    return [l for l in topo.leaf_ids() if all(keep[m] for m in topo.path_to_root(l))]


@pytest.mark.parametrize("K,k", [(2, 1), (4, 2), (3, 1), (2, 2)])
def test_width_modes_counts_and_choice(K, k):
    splits = (0, 2, 3)
    topo, r, logp = _random_case(5, K, splits, seed=K * 10 + k)
    rbar = credit.fuse_rewards(topo, r, logp, 0.0)
    keep = credit.width_keep(topo, rbar, credit.WIDTH_PER_SPLIT_TOPK, k)
    assert len(_kept_leaves(topo, keep)) == k ** len(splits)
    # brute force: a node is kept iff at every split ancestor (itself included) it ranks < k among siblings
    for n in range(1, topo.nodes):
        ok = True
        for m in topo.path_to_root(n)[:-1]:
            p = int(topo.parent[m])
            if int(topo.depth[p]) in splits:
                sib = topo.children(p)
                rank = sum(1 for q in sib if (rbar[q] > rbar[m]) or (rbar[q] == rbar[m] and q < m))
                ok &= rank < k
        assert keep[n] == int(ok)
    last = credit.width_keep(topo, rbar, credit.WIDTH_LAST_SPLIT_TOPK, k)
    assert len(_kept_leaves(topo, last)) == topo.leaves // K * k
    assert np.all(last[:topo.offset[4]] == 1)       # nothing above the last split is touched
    assert np.all(credit.width_keep(topo, rbar, credit.WIDTH_NONE, 0) == 1)


def test_parent_top1_roughly_halves_and_keeps_the_better_child():
    topo, r, _ = _random_case(16, 2, (0, 3, 6, 9), seed=1)
    rbar = credit.fuse_rewards(topo, r, None, 0.0)
    keep = credit.width_keep(topo, rbar, credit.WIDTH_LAST_SPLIT_TOPK, 1)
    assert len(_kept_leaves(topo, keep)) == 8
    for p in topo.level(9):
        a, b = topo.children(p)
        assert keep[a] + keep[b] == 1 and keep[a] == int(rbar[a] >= rbar[b])


def test_ties_prefer_the_lower_branch():
    topo = tree.build_topology(2, 3, (0,))
    rbar = credit.fuse_rewards(topo, np.array([1.0, 1.0, 1.0]), None, 0.0)
    keep = credit.width_keep(topo, rbar, credit.WIDTH_PER_SPLIT_TOPK, 2)
    assert list(keep[1:4]) == [1, 1, 0]
    ex = credit.width_keep(topo, rbar, credit.WIDTH_EXTREME_B, 1)
    assert _kept_leaves(topo, ex) == [topo.offset[2]]          # best = worst = leaf 0


def test_extreme_b():
    topo, r, _ = _random_case(6, 2, (0, 1, 2, 3), seed=9)
    rbar = credit.fuse_rewards(topo, r, None, 0.0)
    first = topo.offset[topo.T]
    for b in (1, 3, 8, 20):
        keep = credit.width_keep(topo, rbar, credit.WIDTH_EXTREME_B, b)
        kept = _kept_leaves(topo, keep)
        assert len(kept) == min(2 * b, topo.leaves)
        order = np.argsort(-r, kind="stable")
        expect = set(order[:b]) | set(order[::-1][:b])
        assert set(l - first for l in kept) == expect
        # kept set = union of root paths
        nodes = set(m for l in kept for m in topo.path_to_root(l))
        assert set(np.nonzero(keep)[0]) == nodes


def test_depth_mask_and_final_mask():
    topo, r, _ = _random_case(16, 2, (0, 3, 6, 9), seed=2)
    rbar = credit.fuse_rewards(topo, r, None, 0.0)
    pruned = [2, 5, 9, 15]
    dk = credit.depth_keep(topo, pruned)
    assert int((dk == 0).sum()) == sum(topo.width[i + 1] for i in pruned)
    m = credit.gradient_mask(topo, rbar, credit.WIDTH_PER_SPLIT_TOPK, 2, pruned)
    assert m[0] == 0 and int(m.sum()) == topo.edges - sum(topo.width[i + 1] for i in pruned)
    m2 = credit.gradient_mask(topo, rbar, credit.WIDTH_NONE, 0, (), ignore_last_step=True)
    assert int(m2.sum()) == topo.edges - topo.leaves
    # pruning never touches the signals it is computed from
    before = rbar.copy()
    credit.gradient_mask(topo, rbar, credit.WIDTH_EXTREME_B, 2, pruned, True)
    assert np.array_equal(before, rbar)


def test_sliding_window_schedule():
    """Window of size 4 starting at the last split point, one step deeper every 30 iterations."""
    assert credit.depth_window(0, 9) == [9, 10, 11, 12]
    assert credit.depth_window(29, 9) == [9, 10, 11, 12]
    assert credit.depth_window(30, 9) == [10, 11, 12, 13]
    assert credit.depth_window(95, 9, stop=16) == [12, 13, 14, 15]
    assert credit.depth_window(3000, 9, stop=16) == [12, 13, 14, 15]
    assert credit.depth_window(61, 10, size=2, every=20) == [13, 14]


def test_grpo_objective_equals_library_clipped_surrogate():
    """Eq. 5 against the clipped surrogate composed from torch primitives, and its textbook cases."""
    import torch
    topo, r, logp_old = _random_case(6, 2, (0, 2, 4), seed=21)
    rng = np.random.default_rng(3)
    logp_new = logp_old + 0.3 * rng.standard_normal(topo.nodes)
    rbar = credit.fuse_rewards(topo, r, logp_old, 1.0)
    adv = credit.depth_advantages(topo, rbar, 1e-6)
    mask = credit.gradient_mask(topo, rbar, credit.WIDTH_PER_SPLIT_TOPK, 1, [1, 4])
    for eps, scale in ((0.2, 1.0), (1e-4, 1.0), (0.1, 3.0)):
        J, terms = credit.grpo_objective(topo, logp_new, logp_old, adv, mask, eps, scale)
        ratio = torch.exp(torch.tensor(scale * (logp_new - logp_old)))
        A = torch.tensor(adv)
        ref = torch.minimum(ratio * A, torch.clamp(ratio, 1 - eps, 1 + eps) * A)
        sel = torch.tensor(mask.astype(bool))
        sel[0] = False
        assert math.isclose(J, float(ref[sel].mean()), rel_tol=1e-12, abs_tol=1e-15)
        assert np.allclose(terms[mask.astype(bool)], ref[sel].numpy(), rtol=1e-12)
        assert np.all(terms[~mask.astype(bool)] == 0)
    # new policy == old policy: rho = 1, J = mean advantage over the edge set; over ALL edges the depth-wise
    # standardisation makes every depth sum to zero, so J = 0
    full = np.ones(topo.nodes, dtype=np.uint8)
    J, _ = credit.grpo_objective(topo, logp_old, logp_old, adv, full, 0.2)
    assert abs(J) < 1e-12
    # the three regimes of the clip for one edge
    one = tree.build_topology(1, 1, ())
    for a, dl, eps, expect in ((2.0, 0.5, 0.2, 1.2 * 2.0), (-2.0, -0.5, 0.2, 0.8 * -2.0), (2.0, -0.5, 0.2, math.exp(-0.5) * 2.0),
                               (-2.0, 0.5, 0.2, math.exp(0.5) * -2.0)):
        J, _ = credit.grpo_objective(one, np.array([0.0, dl]), np.zeros(2), np.array([0.0, a]), np.array([0, 1]), eps)
        assert math.isclose(J, expect, rel_tol=1e-12)
    assert credit.grpo_objective(one, np.zeros(2), np.zeros(2), np.ones(2), np.zeros(2, dtype=np.uint8), 0.2)[0] == 0.0


def test_mix_schedule():
    """All branching steps stay SDE; a window of 4 adds further SDE steps and slides every 30 iterations."""
    assert credit.mix_sde_steps(20, (0, 3, 6, 9), 0) == [0, 1, 2, 3, 6, 9]
    assert credit.mix_sde_steps(20, (0, 3, 6, 9), 30 * 5) == [0, 3, 5, 6, 7, 8, 9]
    assert credit.mix_sde_steps(20, (0, 3, 6, 9), 10 ** 6) == [0, 3, 6, 9, 16, 17, 18, 19]
    topo = tree.build_topology(8, 2, (0, 3))
    rbar = np.zeros(topo.nodes)
    m = credit.gradient_mask(topo, rbar, credit.WIDTH_NONE, 0, (), False, sde_steps=[0, 3, 5])
    for n in range(1, topo.nodes):
        assert m[n] == int(topo.depth[n] - 1 in (0, 3, 5))


# ---------------------------------------------------------------------------------------------- ESS of the fusion weights
def test_fusion_ess_special_cases_and_bounds():
    """Appendix "Reward Fusion": ESS = (sum w)^2 / sum w^2.  beta = 0 -> the number of descendant leaves; equal edge
    log-probs -> the same for any beta; a two-leaf node with path probabilities (p, 1-p) at beta = 1 -> 1/(p^2+(1-p)^2);
    one overwhelming leaf -> 1; always 1 <= ESS <= |L(n)|."""
    topo = tree.build_topology(5, 3, (0, 2, 3))
    n_leaves = np.array([len(topo.descendant_leaves(n)) for n in range(topo.nodes)], dtype=np.float64)
    rng = np.random.default_rng(5)
    logp = rng.normal(-1.0, 0.7, size=topo.nodes)
    assert np.allclose(credit.fusion_ess(topo, logp, 0.0), n_leaves)
    assert np.allclose(credit.fusion_ess(topo, np.full(topo.nodes, -0.3), 2.5), n_leaves)
    for beta in (0.5, 1.0, 4.0):
        ess = credit.fusion_ess(topo, logp, beta)
        assert np.all(ess >= 1.0 - 1e-12) and np.all(ess <= n_leaves + 1e-9)
        assert np.allclose(ess[topo.offset[topo.T]:], 1.0)               # a leaf is its own only descendant
    # two leaves under one parent, probabilities p and 1 - p
    t2 = tree.build_topology(1, 2, (0,))
    p = 0.8
    lp = np.array([0.0, math.log(p), math.log(1 - p)])
    assert credit.fusion_ess(t2, lp, 1.0)[0] == pytest.approx(1.0 / (p * p + (1 - p) * (1 - p)), rel=1e-12)
    # textbook form on explicit normalised weights
    t3 = tree.build_topology(2, 2, (0, 1))
    lp3 = rng.normal(size=t3.nodes)
    s = np.array([credit.path_logp(t3, lp3, 0, l) for l in t3.leaf_ids()])
    w = special.softmax(1.3 * s)
    assert credit.fusion_ess(t3, lp3, 1.3)[0] == pytest.approx(1.0 / np.sum(w ** 2), rel=1e-12)
    # one leaf overwhelmingly likely
    lp_dom = np.full(t3.nodes, -50.0)
    leaf = t3.leaf_ids()[2]
    m = leaf
    while m > 0:
        lp_dom[m] = 0.0
        m = int(t3.parent[m])
    assert credit.fusion_ess(t3, lp_dom, 1.0)[0] == pytest.approx(1.0, abs=1e-12)
