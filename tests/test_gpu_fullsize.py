"""Full-size parity in the launch configuration the benchmark times: the video-shaped tree
(21x60x104 tokens x 16 channels, 111 nodes, closed-form velocity) is small enough for the
oracle to compute whole, so every latent element, every log-prob, every reward, advantage and
mask of the full workload is compared."""
import numpy as np
import pytest
import torch

from oracle import credit, rewards
from oracle import tree as otree
from workloads import CONFIGS, make_inputs

from test_gpu_parity import LATENT_TOL, LOGP_TOL, B, adv_close, assert_table, f32, oracle_rollout  # noqa: F401

pytestmark = pytest.mark.gpu


def test_video_config_whole_workload(B):
    from paper_2509_06040_b200.session import TreeSession
    w = CONFIGS["video"]
    inp = make_inputs(w)
    s = TreeSession(w)
    s.upload_inputs(inp)
    s.run_all()
    torch.cuda.synchronize()
    B.tree_sync_status(s.tree)
    topo, lat, logp = oracle_rollout(w, inp, 1)
    assert_table(s, topo, 1)
    got = s.latents.cpu().numpy()
    worst = 0.0
    for n in range(topo.nodes):
        worst = max(worst, float(np.abs(got[0, n] - lat[0, n]).max()))
    assert worst <= LATENT_TOL, worst
    assert np.abs(s.logp.cpu().numpy() - logp).max() <= LOGP_TOL
    # siblings share their prefix: there is one stored row per node, and children of a split differ
    for p in topo.level(5):
        a, b = topo.children(p)
        assert not np.array_equal(got[0, a], got[0, b])
    r = np.array([rewards.neg_mse(lat[0][l], inp.target[0]) for l in topo.leaf_ids()])
    got_r = s.leaf_r.cpu().numpy()[0]
    assert np.abs(got_r - r).max() <= 1e-6 * np.abs(r).max()
    # reductions, teacher-forced on the oracle's float32 rewards and log-probs
    s.logp.copy_(torch.from_numpy(logp.astype(np.float32)))
    s.leaf_r.copy_(torch.from_numpy(r.astype(np.float32)[None]))
    s.fuse_advantage()
    s.prune()
    torch.cuda.synchronize()
    r32 = r.astype(np.float32).astype(np.float64)
    rbar = credit.fuse_rewards(topo, r32, logp[0].astype(np.float32).astype(np.float64), w.beta)
    adv = credit.depth_advantages(topo, rbar, f32(w.eps))
    assert adv_close(s.adv.cpu().numpy()[0], adv)
    rbar32 = s.rbar.cpu().numpy()[0]
    assert np.array_equal(rbar32, rbar.astype(np.float32))
    mask = credit.gradient_mask(topo, rbar32, w.width_mode, w.width_k, (), w.ignore_last_step)
    assert np.array_equal(s.mask.cpu().numpy()[0], mask)
    assert int(mask.sum()) == sum(1 for n in range(1, topo.nodes) if mask[n])
    # top-1 per split keeps exactly one leaf
    assert int(mask[list(topo.leaf_ids())].sum()) == 1


@pytest.mark.parametrize("name,depth", [("image", 0), ("image", 10), ("image_batch", 10), ("group", 12)])
def test_mlp_stage_full_size_sampled(B, name, depth):
    """The MLP velocity stage at the benchmark's sizes and launch shapes: the root level of the single image tree (16
    tiles, cut 8 ways along the hidden dimension), its widest level (254 tiles on 148 SMs), the widest level of the
    32-tree batch (8100 tiles) and of the 8-tree group workload.  The frontier is filled with seeded normal latents; a
    sample of tokens (tile heads and tails, tree and node boundaries, the ragged last tile, random ones) is compared with
    the oracle's bf16-emulating MLP, token by token."""
    from oracle import mlp
    from paper_2509_06040_b200.session import TreeSession
    w = CONFIGS[name]
    inp = make_inputs(w)
    s = TreeSession(w)
    s.upload_inputs(inp)
    s.init()
    s.v.zero_()
    for i in range(depth):                       # grow the tree to the depth under test; the latents are replaced below
        B.tree_step(s.tree, 1 if i in w.splits else 0, s.v)
    widths, offs = B.tree_levels(s.tree)
    W, off = widths[depth], offs[depth]
    rng = np.random.default_rng([7, depth, w.n_trees])
    z = rng.standard_normal((w.n_trees, W, w.D), dtype=np.float32)
    s.latents[:, off:off + W].copy_(torch.from_numpy(z))
    s.v.fill_(float("nan"))
    B.velocity_mlp(s.tree, s.packed, w.hidden, s.v)
    torch.cuda.synchronize()
    B.tree_sync_status(s.tree)
    n_tok = w.n_trees * W * w.tokens
    got = s.v.view(-1)[:n_tok * 64].view(n_tok, 64)
    zt = z.reshape(n_tok, 64)
    per_tree = W * w.tokens
    picks = set(range(0, 130)) | set(range(n_tok - 130, n_tok)) | {int(x) for x in rng.integers(0, n_tok, 400)}
    for t in range(1, min(w.n_trees, 3)):        # around tree boundaries
        picks |= set(range(t * per_tree - 3, t * per_tree + 3))
    for j in range(1, min(W, 3)):                # around node boundaries
        picks |= set(range(j * w.tokens - 3, j * w.tokens + 3))
    for tile in (1, 2, (n_tok // 128) // 2):     # heads and tails of some tiles
        picks |= set(range(tile * 128 - 2, tile * 128 + 2))
    idx = np.array(sorted(p for p in picks if 0 <= p < n_tok))
    ref = mlp.mlp_velocity(zt[idx], inp.W1, inp.W2)
    out = got[torch.from_numpy(idx).cuda()].cpu().numpy()
    rms = float(np.sqrt(np.mean(ref.astype(np.float64) ** 2)))
    d = np.abs(out - ref)
    print(f"{name} depth {depth}: worst |d|/rms(v) = {d.max() / rms:.4f}, rms |d|/rms(v) = {np.sqrt(np.mean(d ** 2)) / rms:.4f}")
    assert np.all(d <= 2e-2 * np.abs(ref) + 2e-2 * rms), float(d.max() / rms)
    large = np.abs(ref) >= rms
    assert np.all(d[large] <= 2e-2 * np.abs(ref[large]))      # plain relative bound where the output is not small
    assert not torch.isnan(got).any()            # every token of the frontier was written


@pytest.mark.parametrize("name,depth", [("image_batch", 9), ("image_batch", 10), ("group", 12)])
def test_step_kernel_full_size_sampled_rows(B, name, depth):
    """tree_step with a supplied velocity at the benchmark's widest launches (a split step and a non-split one of the
    32-tree batch, the 64-wide level of the group workload): frontier latents and velocities are seeded normals, and for
    a sample of (tree, parent) pairs - first, last, around the middle - every element of every child row and the
    children's log-probs are compared with the oracle's Euler-Maruyama step (Eq. 2) on the same inputs."""
    from oracle import philox, sde
    from paper_2509_06040_b200.session import TreeSession
    w = CONFIGS[name]
    s = TreeSession(w)
    s.upload_inputs(make_inputs(w))
    s.init()
    s.v.zero_()
    for i in range(depth):
        B.tree_step(s.tree, 1 if i in w.splits else 0, s.v)
    widths, offs = B.tree_levels(s.tree)
    W, off = widths[depth], offs[depth]
    rng = np.random.default_rng([11, depth, w.n_trees])
    z = rng.standard_normal((w.n_trees, W, w.D), dtype=np.float32)
    v = rng.standard_normal((w.n_trees, W, w.D), dtype=np.float32)
    s.latents[:, off:off + W].copy_(torch.from_numpy(z))
    v_dev = s.v.view(-1)[:z.size].view(z.shape)
    v_dev.copy_(torch.from_numpy(v))
    split = depth in w.splits
    B.tree_step(s.tree, 1 if split else 0, v_dev)
    # the step's own log-prob sums are completed by the next call on the stream: here the recompute under the same
    # velocity, which must give the same numbers (rho = 1)
    again = torch.zeros_like(s.logp)
    B.tree_logprob(s.tree, depth, v_dev, again)
    torch.cuda.synchronize()
    B.tree_sync_status(s.tree)
    widths, offs = B.tree_levels(s.tree)
    off_c, fan = offs[depth + 1], (w.K if split else 1)
    grid = w.t_grid().astype(np.float64)
    t, h, sigma = float(grid[depth]), float(grid[depth] - grid[depth + 1]), f32(w.sigma)
    g = sde.noise_scale(sigma, h)
    logp = s.logp.cpu().numpy()
    for tree, j in ((0, 0), (w.n_trees - 1, W - 1), (w.n_trees // 2, W // 2), (1, 1)):
        mean = sde.em_mean(z[tree, j].astype(np.float64), v[tree, j].astype(np.float64), t, h, sigma)
        for b in range(fan):
            c = off_c + j * fan + b
            eta = philox.node_noise(w.seed, tree * s.nodes_cap + c, depth, philox.TAG_INNOV, w.D)
            child = (mean + g * eta).astype(np.float32)           # the workloads run with independent children (s = inf)
            got = s.latents[tree, c].cpu().numpy()
            assert np.abs(got - child).max() <= LATENT_TOL, (tree, j, b)
            assert abs(logp[tree, c] - sde.transition_logp(child, mean, g)) <= LOGP_TOL
            assert abs(float(again[tree, c]) - sde.transition_logp(child, mean, g)) <= LOGP_TOL
    tab = s.node_table.cpu().numpy().reshape(4, w.n_trees, s.nodes_cap)
    assert np.array_equal(tab[0, 0, off_c:off_c + W * fan], off + np.arange(W * fan) // fan)
    assert np.all(tab[1, :, off_c:off_c + W * fan] == depth + 1)


def test_cosine_reward_at_the_image_size_every_row(B):
    """The cosine leaf reward of the 32-tree image batch in the launch configuration the benchmark times: 512 leaf rows
    of 129 600 elements (32 chunks of 4096 per row, exactly one lane-stride of the finish kernel's sum) filled with
    seeded normals, every row against the oracle (Algorithm 1, "Evaluate rewards for leaves")."""
    from paper_2509_06040_b200.session import TreeSession
    w = CONFIGS["image_batch"]
    inp = make_inputs(w)
    s = TreeSession(w)
    s.upload_inputs(inp)
    s.init()
    s.v.zero_()
    for i in range(w.T):                          # grow the tree; the leaf rows are replaced below
        B.tree_step(s.tree, 1 if i in w.splits else 0, s.v)
    widths, offs = B.tree_levels(s.tree)
    L, off = widths[w.T], offs[w.T]
    assert L == w.leaves == 16
    rng = np.random.default_rng([13, w.n_trees])
    z = (0.7 * rng.standard_normal((w.n_trees, L, w.D), dtype=np.float32) + 0.05 * inp.target[:, None, :]).astype(np.float32)
    s.latents[:, off:off + L].copy_(torch.from_numpy(z))
    s.rewards()                                   # seeded draw + 0.1 cos(z_leaf, target)
    first = s.leaf_r.clone()
    s.rewards()
    torch.cuda.synchronize()
    B.tree_sync_status(s.tree)
    assert torch.equal(first, s.leaf_r)           # fixed summation order: the same bits on a second run
    got = s.leaf_r.cpu().numpy()
    worst = 0.0
    for t in range(w.n_trees):
        for q in range(L):
            ref = float(inp.reward_draws[t, q]) + 0.1 * rewards.cosine(z[t, q], inp.target[t])
            worst = max(worst, abs(got[t, q] - ref) / max(1.0, abs(ref)))
    assert worst <= 1e-6, worst
    # and the -MSE mode on the same rows
    B.leaf_reward_mse(s.tree, s.target, s.leaf_r)
    torch.cuda.synchronize()
    got = s.leaf_r.cpu().numpy()
    for t in range(w.n_trees):
        for q in range(L):
            ref = rewards.neg_mse(z[t, q], inp.target[t])
            assert abs(got[t, q] - ref) <= 1e-6 * max(1.0, abs(ref))


@pytest.mark.parametrize("name", ["image_batch", "group"])
def test_reductions_with_the_batched_configs_tree_counts(B, name):
    """Reward fusion, depth-wise advantages and the pruning masks launched as the batched configurations launch them -
    32 trees with top-2 per split and the seeded 4 of 16 pruned steps; 8 trees of 765 nodes with the mixture rewards -
    every tree against the oracle (Eq. 3, Eq. 4, "Pruning Strategies").  The reductions never look at the latents, so
    the trees are grown with 16 elements per node; rewards and log-probs are teacher-forced in float32."""
    from paper_2509_06040_b200.session import TreeSession
    cfg = CONFIGS[name]
    inp_full = make_inputs(cfg.scaled(tokens=1, channels=64))       # the per-leaf reward draws and pruned steps of the config
    w = cfg.scaled(name=name + "_reductions", tokens=4, channels=4, velocity="linear", reward="neg_mse_mu")
    s = TreeSession(w)
    s.upload_inputs(make_inputs(w))
    s.rollout()
    s.pruned_steps = tuple(int(x) for x in inp_full.pruned_steps)
    topo = otree.build_topology(w.T, w.K, w.splits)
    assert topo.nodes == cfg.nodes
    rng = np.random.default_rng([17, w.n_trees])
    r = inp_full.reward_draws.astype(np.float32)
    lp = (-0.9 + 0.2 * rng.standard_normal((w.n_trees, topo.nodes))).astype(np.float32)
    lp[:, 0] = 0
    s.logp.copy_(torch.from_numpy(lp))
    s.leaf_r.copy_(torch.from_numpy(r))
    for beta in (w.beta, 1.0):
        B.tree_fuse_advantage(s.tree, s.leaf_r, beta, 1.0, f32(w.eps), f32(w.adv_clip))
        s.prune()
        torch.cuda.synchronize()
        B.tree_sync_status(s.tree)
        got_rbar, got_adv, got_mask = s.rbar.cpu().numpy(), s.adv.cpu().numpy(), s.mask.cpu().numpy()
        for t in range(w.n_trees):
            rbar = credit.fuse_rewards(topo, r[t].astype(np.float64), lp[t].astype(np.float64), beta)
            adv = credit.depth_advantages(topo, rbar, f32(w.eps))
            assert np.abs(got_rbar[t] - rbar).max() <= 1e-6 * max(1.0, np.abs(rbar).max()), t
            assert adv_close(got_adv[t], adv), t
            mask = credit.gradient_mask(topo, got_rbar[t], w.width_mode, w.width_k, s.pruned_steps, w.ignore_last_step)
            assert np.array_equal(got_mask[t], mask), t
    if name == "image_batch":
        assert len(s.pruned_steps) == 4
        # top-2 of 2 children keeps every child: the mask is exactly the depth mask (reading R8 of the configs)
        depth_only = credit.gradient_mask(topo, got_rbar[0], 0, 0, s.pruned_steps, False)
        assert np.array_equal(got_mask[0], depth_only)
