"""Pins for oracle/tree.py: node counts against the NFE and leaf counts the paper prints,
and the structure against a brute-force construction."""
import os

import numpy as np
import pytest

from oracle import tree
from workloads import CONFIGS


def _rows(golden_dir, name):
    for line in open(os.path.join(golden_dir, name)):
        if line.startswith("#") or not line.strip():
            continue
        yield line.split()


def test_nfe_matches_printed_table(golden_dir):
    n = 0
    for splits, printed in _rows(golden_dir, "nfe_table1.txt"):
        topo = tree.build_topology(20, 2, [int(x) for x in splits.split(",")])
        nfe = tree.nfe_per_sample(topo)
        # the paper prints two decimals, truncated (13.6875 -> 13.68) or rounded (9.4375 -> 9.44)
        assert abs(nfe - float(printed)) < 0.01
        n += 1
    assert n == 3
    assert tree.build_topology(20, 2, (0, 3, 6, 9)).nodes == 219


def test_leaf_counts_match_paper(golden_dir):
    for K, n_splits, leaves in _rows(golden_dir, "leaf_counts.txt"):
        topo = tree.build_topology(20, int(K), range(0, 3 * int(n_splits), 3))
        assert topo.leaves == int(leaves)


@pytest.mark.parametrize("name,nodes,edges,evals,leaves", [
    ("toy", 13, 12, 9, 4), ("image", 155, 154, 139, 16), ("group", 765, 764, 701, 64), ("video", 111, 110, 103, 8)])
def test_workload_counts(name, nodes, edges, evals, leaves):
    w = CONFIGS[name]
    topo = tree.build_topology(w.T, w.K, w.splits)
    assert (topo.nodes, topo.edges, topo.model_evals, topo.leaves) == (nodes, edges, evals, leaves)
    assert (w.nodes, w.node_steps, w.model_evals, w.leaves) == (nodes, edges, evals, leaves)
    assert tree.savings_vs_sequential(topo) == evals / (leaves * w.T)


def _brute_tree(T, K, splits):
    """Grow the tree as explicit python objects, breadth first."""
    nodes = [dict(parent=-1, depth=0, split=-1, branch=0)]
    frontier = [0]
    for i in range(T):
        nxt = []
        for p in frontier:
            for b in range(K if i in splits else 1):
                nodes.append(dict(parent=p, depth=i + 1,
                                  split=i if i in splits else nodes[p]["split"],
                                  branch=b if i in splits else nodes[p]["branch"]))
                nxt.append(len(nodes) - 1)
        frontier = nxt
    return nodes


@pytest.mark.parametrize("T,K,splits", [(4, 2, (0, 2)), (5, 3, (1, 4)), (6, 4, (0, 1, 5)), (3, 2, ()), (3, 2, (0, 1, 2))])
def test_table_equals_brute_force(T, K, splits):
    topo = tree.build_topology(T, K, splits)
    ref = _brute_tree(T, K, splits)
    assert topo.nodes == len(ref)
    for n, r in enumerate(ref):
        assert (topo.parent[n], topo.depth[n], topo.split_step[n], topo.branch_id[n]) == \
               (r["parent"], r["depth"], r["split"], r["branch"])
        for c in topo.children(n):
            assert ref[c]["parent"] == n
    # L(n) by walking down equals the leaves whose root path passes through n
    for n in range(topo.nodes):
        via_paths = [l for l in topo.leaf_ids() if n in topo.path_to_root(l)]
        assert topo.descendant_leaves(n) == via_paths


def test_prefix_sharing():
    """Two leaves share exactly the nodes above their lowest common split."""
    topo = tree.build_topology(16, 2, (0, 3, 6, 9))
    leaves = list(topo.leaf_ids())
    for a in leaves[:4]:
        for b in leaves:
            pa, pb = topo.path_to_root(a)[::-1], topo.path_to_root(b)[::-1]
            common = sum(1 for x, y in zip(pa, pb) if x == y)
            assert pa[:common] == pb[:common] and (a == b or pa[common] != pb[common])
            if a != b:
                # they diverge right after a split step
                assert int(topo.depth[pa[common]]) - 1 in topo.splits
