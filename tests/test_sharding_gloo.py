"""The N > 1 path on CPU: two gloo ranks each take a contiguous shard of the trees (the path has no exchange step),
draw their inputs and noise by GLOBAL tree index, and together reproduce the single-process result bit for bit; the
timing reduction the benchmark uses (max over ranks) is exercised as well.  The per-rank compute is the oracle here -
the host logic under test is the sharding, the id bookkeeping and the reductions."""
import math
import os

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from workloads import Workload, make_inputs, shard_trees

W = Workload(name="shard", n_trees=3, tokens=8, channels=4, T=3, K=2, splits=(0, 2), sigma=0.3,
             velocity="linear", reward="neg_mse_mu")


def _rollout_shard(first, count):
    from oracle import sde, tree
    topo = tree.build_topology(W.T, W.K, W.splits)
    grid = W.t_grid().astype(np.float64)
    inp = make_inputs(W.scaled(n_trees=count), tree_base=first)
    out = []
    for t in range(count):
        mu = inp.mu[t].astype(np.float64)
        lat, logp = sde.rollout(topo, W.D, grid, float(np.float32(W.sigma)), math.inf, W.seed,
                                lambda z, i, p: sde.linear_velocity(z.astype(np.float64), float(grid[i]), mu, 0.5),
                                tree_id=first + t, nodes_cap=topo.nodes)
        out.append((lat, logp))
    return out


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    first, count = shard_trees(W.n_trees, rank, world)
    mine = _rollout_shard(first, count)
    gathered = [None] * world
    dist.all_gather_object(gathered, (first, mine))
    t = torch.tensor([10.0 + rank], dtype=torch.float64)        # a per-rank "elapsed time"
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.barrier()
    if rank == 0:
        q.put((gathered, float(t.item())))
    dist.destroy_process_group()


def test_shards_cover_all_trees_once():
    for total in (1, 3, 8, 32, 33):
        for world in (1, 2, 4, 8):
            spans = [shard_trees(total, r, world) for r in range(world)]
            ids = [t for first, n in spans for t in range(first, first + n)]
            assert ids == list(range(total))
            assert max(n for _, n in spans) - min(n for _, n in spans) <= 1


def test_two_gloo_ranks_reproduce_the_single_process_trees():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    gathered, tmax = q.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert tmax == 11.0
    whole = _rollout_shard(0, W.n_trees)
    seen = {}
    for first, shard in gathered:
        for k, (lat, logp) in enumerate(shard):
            seen[first + k] = (lat, logp)
    assert sorted(seen) == [0, 1, 2]
    for t in range(W.n_trees):
        assert np.array_equal(seen[t][0], whole[t][0]) and np.array_equal(seen[t][1], whole[t][1])
    assert not np.array_equal(whole[0][0], whole[1][0])
