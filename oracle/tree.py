"""Rollout-tree topology for the oracle (test infrastructure).

"Preliminaries" of the Branch Rollout section: depth T = number of denoising
steps, width w = number of leaves, branching steps B, branching factor K.
Step index i counts from the noise end (t_0 = 1 is the noisiest state): the
paper calls the preset (0,3,6,9) "early splits", so step 0 is the first
transition.  A split at step i means the transition i -> i+1 produces K
children per live node (Eq. 2); any other step produces one child
(Algorithm 1, "Branch into K children" / "Single-step denoising").

Nodes are stored in level order: depth d occupies local indices
offset[d] .. offset[d] + width[d] - 1, and the children of the j-th node of
depth d are the nodes j*K + b (split) or j (no split) of depth d + 1.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Sequence

import numpy as np


@dataclass
class Topology:
    T: int
    K: int
    splits: tuple
    width: List[int]          # width[d], d = 0..T
    offset: List[int]         # offset[d], d = 0..T+1 (offset[T+1] = node count)
    parent: np.ndarray        # [nodes] local parent index, -1 for the root
    depth: np.ndarray         # [nodes]
    split_step: np.ndarray    # [nodes] step of the most recent split on the path to the node, -1 if none
    branch_id: np.ndarray     # [nodes] branch index b taken at that split, 0 if none

    @property
    def nodes(self) -> int:
        return self.offset[-1]

    @property
    def leaves(self) -> int:
        return self.width[-1]

    @property
    def edges(self) -> int:
        """Node-steps: one per non-root node."""
        return self.nodes - 1

    @property
    def model_evals(self) -> int:
        """Velocity evaluations: one per parent, shared by its children."""
        return self.nodes - self.leaves

    def fanout(self, step: int) -> int:
        return self.K if step in self.splits else 1

    def children(self, n: int) -> List[int]:
        d = int(self.depth[n])
        if d == self.T:
            return []
        j = n - self.offset[d]
        f = self.fanout(d)
        return [self.offset[d + 1] + j * f + b for b in range(f)]

    def level(self, d: int) -> range:
        return range(self.offset[d], self.offset[d] + self.width[d])

    def leaf_ids(self) -> range:
        return self.level(self.T)

    def descendant_leaves(self, n: int) -> List[int]:
        """L(n) of Eq. 3, by walking down from n."""
        front = [n]
        for _ in range(int(self.depth[n]), self.T):
            front = [c for m in front for c in self.children(m)]
        return front

    def path_to_root(self, n: int) -> List[int]:
        out = [n]
        while self.parent[out[-1]] >= 0:
            out.append(int(self.parent[out[-1]]))
        return out


def build_topology(T: int, K: int, splits: Sequence[int]) -> Topology:
    splits = tuple(sorted(int(s) for s in splits))
    assert all(0 <= s < T for s in splits), "split steps must lie in 0..T-1"
    width, offset = [1], [0]
    for i in range(T):
        width.append(width[-1] * (K if i in splits else 1))
    for d in range(T + 1):
        offset.append(offset[-1] + width[d])
    n = offset[-1]
    parent = np.full(n, -1, dtype=np.int32)
    depth = np.zeros(n, dtype=np.int32)
    split_step = np.full(n, -1, dtype=np.int32)
    branch_id = np.zeros(n, dtype=np.int32)
    for i in range(T):
        f = K if i in splits else 1
        for j in range(width[i]):
            p = offset[i] + j
            for b in range(f):
                c = offset[i + 1] + j * f + b
                parent[c] = p
                depth[c] = i + 1
                if i in splits:
                    split_step[c], branch_id[c] = i, b
                else:
                    split_step[c], branch_id[c] = split_step[p], branch_id[p]
    return Topology(T, K, splits, width, offset, parent, depth, split_step, branch_id)


def nfe_per_sample(topo: Topology) -> float:
    """Average per-sample NFE in the convention of Table 1's caption: the function
    evaluations of the whole tree divided by the number of final samples.  The
    printed values (13.68, 11.56, 9.44 at depth 20) are reproduced when every node
    of the tree, the root included, counts as one evaluation."""
    return topo.nodes / topo.leaves


def savings_vs_sequential(topo: Topology) -> float:
    """Velocity evaluations of the tree over those of `leaves` independent T-step rollouts."""
    return topo.model_evals / (topo.leaves * topo.T)
