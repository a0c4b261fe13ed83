"""Named workload configurations and seeded synthetic inputs.

This module holds no arithmetic of the method: it only names shapes and
schedules and draws the *inputs* (target means, target latents, MLP weights,
leaf-reward draws, pruned-depth subsets) from numpy's seeded generators.  The
noise the method itself draws (root latent, branch noise) is not made here: it
comes from the counter-based generator that each implementation builds from
the published definition.

Shapes follow the paper's workloads: a 720x720 image with a 16-channel VAE and
2x2 patches packs to 2025 tokens x 64 channels (hyper-parameter table,
"Resolution 720x720"); the video latent is 21 frames x 60 x 104 x 16 channels;
K = 2 children at split steps (0,3,6,9) gives 16 leaves ("Implementation
Details").  The paper's prompts, reward models and denoiser weights are not
used: seeded draws of the same shapes stand in for them.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Dict, Tuple

import numpy as np

# width-pruning modes (values are the ones the C header gives)
WIDTH_NONE = 0
WIDTH_PER_SPLIT_TOPK = 1
WIDTH_LAST_SPLIT_TOPK = 2
WIDTH_EXTREME_B = 3

BASE_SEED = 42          # "Random seed 42" (hyper-parameter table)
SAMPLER_SEED = 1223627  # "Sampler seed 1223627" (hyper-parameter table)


@dataclass(frozen=True)
class Workload:
    name: str
    n_trees: int
    tokens: int
    channels: int
    T: int
    K: int
    splits: Tuple[int, ...]
    sigma: float
    velocity: str                 # "linear" | "mlp"
    reward: str                   # "neg_mse_mu" | "neg_mse_target" | "normal_plus_cos" | "mixture"
    s0: float = 0.5               # std of the Gaussian target (linear velocity)
    branch_corr_s: float = float("inf")   # Eq. 2 's'; inf = independent children
    beta: float = 0.0
    eps: float = 1e-6
    adv_clip: float = 0.0         # <= 0: no clipping
    width_mode: int = WIDTH_NONE
    width_k: int = 0
    n_pruned_depths: int = 0
    ignore_last_step: bool = False
    hidden: int = 3072            # MLP hidden width
    seed: int = SAMPLER_SEED
    input_seed: int = BASE_SEED
    description: str = ""

    @property
    def D(self) -> int:
        return self.tokens * self.channels

    def t_grid(self) -> np.ndarray:
        """Uniform grid t_i = 1 - i/T, i = 0..T (float32, as the C-ABI takes it)."""
        return (1.0 - np.arange(self.T + 1, dtype=np.float64) / self.T).astype(np.float32)

    def widths(self):
        w = [1]
        for i in range(self.T):
            w.append(w[-1] * (self.K if i in self.splits else 1))
        return w

    @property
    def leaves(self) -> int:
        return self.widths()[-1]

    @property
    def nodes(self) -> int:
        return int(sum(self.widths()))

    @property
    def node_steps(self) -> int:
        """Edges per tree: one per non-root node."""
        return self.nodes - 1

    @property
    def model_evals(self) -> int:
        """One velocity evaluation per parent node."""
        return int(sum(self.widths()[:-1]))

    def scaled(self, **kw) -> "Workload":
        return replace(self, **kw)


CONFIGS: Dict[str, Workload] = {
    "toy": Workload(
        name="toy", n_trees=1, tokens=16, channels=4, T=4, K=2, splits=(0, 2), sigma=0.3,
        velocity="linear", reward="neg_mse_mu",
        description="1 prompt, 16 tokens x 4 ch, T=4, splits {0,2}, linear velocity, -MSE reward"),
    "image": Workload(
        name="image", n_trees=1, tokens=2025, channels=64, T=16, K=2, splits=(0, 3, 6, 9), sigma=0.3,
        velocity="mlp", reward="normal_plus_cos",
        description="1 prompt, 2025 tokens x 64 ch (720x720), T=16, splits {0,3,6,9}, bf16 MLP velocity"),
    "image_batch": Workload(
        name="image_batch", n_trees=32, tokens=2025, channels=64, T=16, K=2, splits=(0, 3, 6, 9), sigma=0.3,
        velocity="mlp", reward="normal_plus_cos",
        width_mode=WIDTH_PER_SPLIT_TOPK, width_k=2, n_pruned_depths=4,
        description="32 image-shaped trees, top-2 per split, 4 of 16 depths pruned"),
    "group": Workload(
        name="group", n_trees=8, tokens=4096, channels=64, T=20, K=2, splits=(0, 2, 4, 6, 8, 10), sigma=0.5,
        velocity="mlp", reward="mixture",
        description="8 trees, 4096 tokens x 64 ch (1024x1024), T=20, 6 splits (64 leaves), bf16 MLP velocity"),
    "video": Workload(
        name="video", n_trees=1, tokens=21 * 60 * 104, channels=16, T=20, K=2, splits=(0, 5, 10), sigma=0.3,
        velocity="linear", reward="neg_mse_target",
        width_mode=WIDTH_PER_SPLIT_TOPK, width_k=1,
        description="1 prompt, 21x60x104 tokens x 16 ch, T=20, splits {0,5,10}, linear velocity, top-1 per split"),
}
CONFIG_ORDER = ("toy", "image", "image_batch", "group", "video")


@dataclass
class Inputs:
    """Seeded inputs of one workload (numpy, host)."""
    mu: np.ndarray | None = None          # [n_trees][D] float32, Gaussian-target mean (linear velocity)
    target: np.ndarray | None = None      # [n_trees][D] float32, reward target latent
    W1: np.ndarray | None = None          # [channels][hidden] float32 holding bf16-representable values
    W2: np.ndarray | None = None          # [hidden][channels] float32 holding bf16-representable values
    reward_draws: np.ndarray | None = None  # [n_trees][leaves] float32
    pruned_steps: np.ndarray = field(default_factory=lambda: np.zeros(0, np.int32))


def _to_bf16_values(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bf16 (ties to even) and return them as float32.

    Input conditioning only: weights are *stored* as bf16, so both implementations
    receive numbers that bf16 holds exactly.
    """
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32)


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of float32 values that are already bf16-representable."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    assert np.all((u & 0xFFFF) == 0), "values are not bf16-representable"
    return (u >> 16).astype(np.uint16)


def make_inputs(w: Workload, tree_base: int = 0) -> Inputs:
    """Seeded inputs for trees [tree_base, tree_base + n_trees) of workload `w`.

    Per-tree inputs are drawn from a generator keyed by (input_seed, global tree
    index), so a shard of the batch sees the same numbers as the whole batch.
    Weights are shared by all trees.
    """
    out = Inputs()
    D = w.D

    def tree_rng(t, stream):
        return np.random.default_rng([w.input_seed, stream, tree_base + t])

    if w.velocity == "linear":
        out.mu = np.stack([tree_rng(t, 1).standard_normal(D, dtype=np.float32) for t in range(w.n_trees)])
    else:
        g = np.random.default_rng([w.input_seed, 7])
        out.W1 = _to_bf16_values(0.02 * g.standard_normal((w.channels, w.hidden), dtype=np.float32))
        out.W2 = _to_bf16_values(0.02 * g.standard_normal((w.hidden, w.channels), dtype=np.float32))
    if w.reward in ("neg_mse_target", "normal_plus_cos"):
        out.target = np.stack([tree_rng(t, 2).standard_normal(D, dtype=np.float32) for t in range(w.n_trees)])
    if w.reward == "normal_plus_cos":
        out.reward_draws = np.stack(
            [tree_rng(t, 3).standard_normal(w.leaves).astype(np.float32) for t in range(w.n_trees)])
    elif w.reward == "mixture":
        rows = []
        for t in range(w.n_trees):
            g = tree_rng(t, 3)
            comp = g.random(w.leaves) < 0.3
            a = g.standard_normal(w.leaves)
            b = 2.0 + 0.5 * g.standard_normal(w.leaves)
            rows.append(np.where(comp, b, a).astype(np.float32))
        out.reward_draws = np.stack(rows)
    if w.n_pruned_depths > 0:
        g = np.random.default_rng([w.input_seed, 11])
        out.pruned_steps = np.sort(g.choice(w.T, size=w.n_pruned_depths, replace=False)).astype(np.int32)
    return out


def shard_trees(n_trees_total: int, rank: int, world: int) -> Tuple[int, int]:
    """Contiguous block of trees for `rank`: returns (first tree, count).  Trees are
    independent (one per prompt), so sharding needs no exchange step."""
    base, rem = divmod(n_trees_total, world)
    start = rank * base + min(rank, rem)
    return start, base + (1 if rank < rem else 0)
