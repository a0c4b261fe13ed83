"""Out-of-bounds canary: every device buffer the library writes (and the ones it only reads) sits between two guard
bands of 0xFF bytes; after whole passes over ragged shapes - a row length that is not a multiple of any tile, K = 3,
a node table with spare rows, the MLP stage with a partial 128-token tile and the split over the hidden dimension -
plus the log-prob recompute, the effective-sample-size diagnostic and the objective, every guard byte must be
unchanged.  A kernel that writes one element before or past any buffer fails here without faulting the GPU."""
import numpy as np
import pytest
import torch

from workloads import Workload, make_inputs

from test_gpu_parity import B  # noqa: F401

pytestmark = pytest.mark.gpu

GUARD = 4096


class Guarded:
    def __init__(self):
        self.raws = {}

    def make(self, name, like):
        nbytes = like.numel() * like.element_size()
        raw = torch.full((GUARD + ((nbytes + 255) // 256) * 256 + GUARD,), 0xFF, dtype=torch.uint8, device="cuda")
        payload = raw[GUARD:GUARD + nbytes].view(like.dtype).view(like.shape)
        self.raws[name] = (raw, nbytes)
        return payload

    def check(self):
        for name, (raw, nbytes) in self.raws.items():
            assert bool((raw[:GUARD] == 0xFF).all()), f"{name}: bytes before the buffer were written"
            assert bool((raw[GUARD + nbytes:] == 0xFF).all()), f"{name}: bytes past the buffer were written"


def _guarded_session(w, nodes_cap):
    from paper_2509_06040_b200.session import TreeSession
    s = TreeSession(w, nodes_cap=nodes_cap)
    s.upload_inputs(make_inputs(w))
    g = Guarded()
    for name in ("latents", "node_table", "logp", "rbar", "adv", "mask", "scratch", "leaf_r", "v", "mu", "target",
                 "reward_draws"):
        t = getattr(s, name)
        if t is None:
            continue
        fresh = g.make(name, t)
        if name in ("mu", "target", "reward_draws"):
            fresh.copy_(t)
        setattr(s, name, fresh)
    return s, g


@pytest.mark.parametrize("velocity", ["linear", "mlp"])
def test_guard_bands_survive_whole_ragged_passes(B, velocity):
    if velocity == "linear":
        w = Workload(name="guard_lin", n_trees=3, tokens=2125, channels=4, T=5, K=3, splits=(1, 3), sigma=0.3,
                     velocity="linear", reward="neg_mse_target", branch_corr_s=2.0, width_mode=B.WIDTH_PER_SPLIT_TOPK,
                     width_k=1, n_pruned_depths=2)
    else:
        w = Workload(name="guard_mlp", n_trees=3, tokens=171, channels=64, T=4, K=3, splits=(0, 2), sigma=0.3,
                     velocity="mlp", reward="normal_plus_cos", hidden=256, width_mode=B.WIDTH_EXTREME_B, width_k=2)
    s, g = _guarded_session(w, nodes_cap=w.nodes + 5)
    for seed in (3, 4):
        s.run_all(seed=seed)
    extra = g.make("logp_new", s.logp)
    ess = g.make("ess", s.logp)
    terms = g.make("terms", s.logp)
    J = g.make("J", torch.empty(w.n_trees, dtype=torch.float32, device="cuda"))
    fused_guards = None
    if velocity == "linear":
        B.tree_logprob(s.tree, -1, None, extra)
        fused, fused_guards = _guarded_session(w, nodes_cap=w.nodes + 5)      # the one-launch rollout on the same shapes
        fused.fused_rollout = True
        fused.run_all(seed=5)
    else:
        extra.copy_(s.logp)
        B.tree_logprob(s.tree, w.T - 1, s.v, extra)      # the last step's edges under the stored velocities
    B.tree_fusion_ess(s.tree, 1.0, 1.0, ess)
    B.tree_grpo_objective(s.tree, extra, None, 1.0, 0.2, terms, J)
    torch.cuda.synchronize()
    B.tree_sync_status(s.tree)
    g.check()
    if fused_guards is not None:
        fused_guards.check()
    # rows of the pools beyond the tree were never written either (they still hold the fill pattern)
    nodes = w.nodes
    assert bool((s.mask[:, nodes:] == 0xFF).all())
    assert bool(torch.isnan(s.latents[:, nodes:]).all())


def test_guard_bands_around_the_built_in_scratch_entry_point(B):
    rows_like = torch.empty((7, 4100), dtype=torch.float32, device="cuda")
    g = Guarded()
    rows = g.make("rows", rows_like)
    target = g.make("target", rows_like[0])
    out = g.make("out", torch.empty(7, dtype=torch.float32, device="cuda"))
    rows.normal_()
    target.normal_()
    B.reward_mse_static(rows, target, 7, 4100, out)
    torch.cuda.synchronize()
    g.check()
    ref = -((rows.double() - target.double()) ** 2).mean(dim=1)
    assert np.abs(out.cpu().numpy() - ref.cpu().numpy()).max() <= 1e-6 * float(ref.abs().max())
