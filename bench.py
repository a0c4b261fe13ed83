#!/usr/bin/env python
"""Benchmark of the BranchGRPO tree hot path: tree node-steps/s and achieved HBM bandwidth.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

One "step" is one pass of the whole path over one batch of synthetic trees: root init, T x
[velocity, fused tree step], leaf rewards, reward fusion + depth-wise advantages, pruning masks.
A node-step is one edge of a tree (one child latent with its log-prob).  With N > 1 every rank
runs its own shard of trees - the path has no exchange step - and the reported value is all
ranks' node-steps over the slowest rank's time (weak scaling).  `--gpus N` launches the N ranks
itself (one process per GPU under torch.distributed.run) unless it already runs inside such a
launch.

`--impl reference` times the CPU oracle (oracle/), as it stands, on a bounded sample of the same
workload on this machine's host cores; it is a deliberately slow program and a reported baseline.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import re
import socket
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from workloads import CONFIGS, make_inputs  # noqa: E402

METRIC = "tree node-steps/sec and achieved HBM GB/s (% of peak) at 1 B200 vs CPU oracle"
UNIT = "node-steps/s"
L2_BYTES = 126 * 1024 * 1024
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
NOMINAL_HBM_GBS = 8000.0

# DRAM traffic of a kernel from one ncu capture (dram__bytes_read.sum + dram__bytes_write.sum), see profiles/.
# Each entry is the captured launch's bytes and the units (elements / tokens) it processed; the figure reported
# per launch is bytes-per-unit times the units of an average launch of the timed workload (traffic grows in
# proportion to the units).  It is reported only while the kernel's sources still hash to what was captured.
NCU_TRAFFIC = {
    # step kernel: one capture per operand layout (8 B/element with the closed-form velocity, 12 B/element with a velocity buffer)
    "step_kernel_linear": {"bytes": 75.596544e6 + 13.034496e6, "units": 8 * 2096640,             # profiles/step_kernel_video.md
                           "sources": ("tree_step.cu", "philox.cuh"), "shape": "kStep", "source_hash": "d569995ada83"},
    "step_kernel_mlp": {"bytes": 531.169024e6 + 215.974400e6, "units": 32 * 16 * 129600,         # profiles/step_kernel_image_batch.md
                        "sources": ("tree_step.cu", "philox.cuh"), "shape": "kStep", "source_hash": "d569995ada83"},
    "mlp_velocity_kernel": {"bytes": 266.295296e6 + 213.379328e6, "units": 1036800,       # profiles/mlp_velocity_kernel_image_batch.md
                            "sources": ("mlp_velocity.cu",), "shape": "kMlp", "source_hash": "74593cdd150d"},
    "rollout_fused_kernel": {"bytes": 16.816640e6 + 866.172416e6, "units": 110 * 2096640,  # profiles/rollout_fused_kernel_video.md
                             "sources": ("tree_fused.cu", "philox.cuh"), "shape": "kFused", "source_hash": "d4f0707c5632"},
}


def r4(x):
    """Four significant digits: keeps the printed line short."""
    return None if x is None else float(f"{float(x):.4g}")


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        d["_source"] = "measured"
        return d
    d = dict(FALLBACK_PEAKS)
    d["_source"] = "fallback"
    return d


def kernel_source_hash(names, shape=None):
    """Hash of a kernel's own sources and of the lines of internal.h that define its launch shape (constants whose
    name matches `shape`), so that an edit elsewhere in the shared header does not disown a still-valid capture."""
    h = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_2509_06040_b200", "csrc")
    for n in names:
        h.update(open(os.path.join(csrc, n), "rb").read())
    if shape:
        for line in open(os.path.join(csrc, "internal.h")):
            if line.startswith("constexpr") and re.search(shape, line):
                h.update(line.encode())
    return h.hexdigest()[:12]


# ------------------------------------------------------------------------------------------------ algorithmic work
def step_bytes_per_launch(w, n_trees):
    """Algorithmic HBM bytes of each tree_step launch: per parent one read of z (4D) and, with a supplied
    velocity, of v (4D); per child one write (4D); the closed-form velocity's target mean (4D per tree) is
    read once per launch.  Node-table rows, log-probs and reduction partials are negligible and not counted."""
    D, out, width = w.D, [], 1
    for i in range(w.T):
        fan = w.K if i in w.splits else 1
        b = n_trees * width * (4 * D * (2 if w.velocity == "mlp" else 1) + fan * 4 * D)
        if w.velocity == "linear":
            b += n_trees * 4 * D
        out.append(b)
        width *= fan
    return out


def step_children(w):
    """Children written by each tree_step launch of the batch (n_trees * W_{i+1})."""
    out, width = [], 1
    for i in range(w.T):
        width *= (w.K if i in w.splits else 1)
        out.append(w.n_trees * width)
    return out


def ncu_traffic(kernel, units_per_launch):
    """DRAM bytes of an average launch, scaled from the committed ncu capture; None once the kernel has changed."""
    tr = NCU_TRAFFIC[kernel]
    if tr["source_hash"] != kernel_source_hash(tr["sources"], tr.get("shape")):
        return None
    return tr["bytes"] / tr["units"] * units_per_launch


def mlp_flops_per_launch(w, n_trees):
    out, width = [], 1
    for i in range(w.T):
        out.append(n_trees * width * w.tokens * 2 * 2 * w.channels * w.hidden)
        width *= (w.K if i in w.splits else 1)
    return out


# ------------------------------------------------------------------------------------------------ clocks
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(index), f"--query-gpu={self.FIELDS}",
                                       "--format=csv,noheader,nounits", "-lms", "50"], stdout=self.f, stderr=subprocess.DEVNULL)
        except OSError:
            self.p = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.p is None:
            return out
        time.sleep(0.1)
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.p.kill()
        self.f.flush()
        rows = [r.split(",") for r in open(self.f.name).read().strip().splitlines() if r.count(",") >= 7]
        os.unlink(self.f.name)
        if not rows:
            return out
        # median over the samples taken under load (power well above idle), all samples if none qualifies
        power = [float(r[2]) for r in rows]
        loaded = [r for r, pw in zip(rows, power) if pw >= 0.5 * max(power)] or rows
        out["sm_mhz"] = float(np.median([float(r[0]) for r in loaded]))
        out["sm_max_mhz"] = float(rows[0][1])
        out["power_w_max"] = max(power)
        out["samples"] = len(rows)
        out["samples_under_load"] = len(loaded)
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for k, nm in enumerate(names):
            if any("Active" == r[4 + k].strip() for r in rows):
                out["reasons"].append(nm)
        return out


# ------------------------------------------------------------------------------------------------ ranks
def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def spawn_ranks(n, argv):
    """Re-runs this script as n ranks on this node (one per GPU) under torch.distributed.run and returns its exit code."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}", "--master-addr", "127.0.0.1",
           "--master-port", str(free_port()), os.path.abspath(__file__)] + list(argv)
    return subprocess.call(cmd)


class RankGroup:
    """The only cross-rank plumbing of the benchmark: a barrier and a MAX over ranks of a measured time.  The path itself
    has no exchange step (every rank owns whole trees)."""

    def __init__(self, backend, device=None):
        import torch
        self.torch = torch
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.rank = int(os.environ.get("RANK", "0"))
        self.local = int(os.environ.get("LOCAL_RANK", "0"))
        self.device = device
        self.dist = None
        if self.world > 1:
            import torch.distributed as dist
            os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
            kw = {"device_id": device} if (backend == "nccl" and device is not None) else {}
            dist.init_process_group(backend, **kw)
            self.dist = dist

    def barrier(self):
        if self.dist is not None:
            self.dist.barrier()

    def max(self, x: float) -> float:
        if self.dist is None:
            return float(x)
        t = self.torch.tensor([x], dtype=self.torch.float64, device=self.device if self.device is not None else "cpu")
        self.dist.all_reduce(t, op=self.dist.ReduceOp.MAX)
        return float(t.item())

    def close(self):
        if self.dist is not None:
            self.dist.barrier()
            self.dist.destroy_process_group()


# ------------------------------------------------------------------------------------------------ oracle timing
def _oracle_slice(job):
    """One worker's share of an oracle pass: the rollout of a slice of one tree's latent row - elements for the
    closed-form velocity, whole tokens for the MLP.  Runs in a spawned process with numpy's BLAS on one thread.
    Returns (log-probs of the slice, leaf latents of the slice)."""
    name, start, count = job
    try:
        from threadpoolctl import threadpool_limits
        threadpool_limits(1)
    except Exception:
        pass
    from oracle import mlp, sde
    from oracle import tree as otree
    w = CONFIGS[name]
    inp = make_inputs(w.scaled(n_trees=1))
    topo = otree.build_topology(w.T, w.K, w.splits)
    grid = w.t_grid().astype(np.float64)
    sig, s0 = float(np.float32(w.sigma)), float(np.float32(w.s0))
    if w.velocity == "linear":
        mu = inp.mu[0][start:start + count].astype(np.float64)
        vel = lambda z, i, p: sde.linear_velocity(z.astype(np.float64), float(grid[i]), mu, s0)
    else:
        n_tok = count // w.channels
        vel = lambda z, i, p: mlp.mlp_velocity(z.reshape(n_tok, w.channels), inp.W1, inp.W2).reshape(-1)
    lat, logp = sde.rollout(topo, count, grid, sig, w.branch_corr_s, w.seed, vel, elem_start=start)
    return logp, lat[list(topo.leaf_ids())]


def oracle_pass(w, fraction, workers):
    """One pass of the oracle over the first `fraction` of one tree's latent row, the row split over `workers`
    processes (1: in this process).  Returns (seconds, node-steps/s of a full tree after linear scaling by the row
    fraction, description).  Log-probs of a partial row are partial sums; they only feed the timing."""
    from oracle import credit, rewards
    from oracle import tree as otree
    topo = otree.build_topology(w.T, w.K, w.splits)
    unit = 4 if w.velocity == "linear" else w.channels
    total_units = w.D // unit
    workers = max(1, min(workers, total_units))          # never more processes than slices of the row
    n_units = min(total_units, max(workers, int(total_units * fraction)))
    bounds = np.linspace(0, n_units, workers + 1).astype(int)
    jobs = [(w.name, int(bounds[k]) * unit, int(bounds[k + 1] - bounds[k]) * unit) for k in range(workers)]
    inp = make_inputs(w.scaled(n_trees=1))
    if workers == 1:
        t0 = time.perf_counter()
        res = [_oracle_slice(jobs[0])]
    else:
        import multiprocessing as mp
        with mp.get_context("spawn").Pool(workers) as pool:      # spawn: this process may already hold a CUDA context
            pool.map(_noop, range(4 * workers))                  # interpreter and numpy start-up stay outside the timing
            t0 = time.perf_counter()
            res = pool.map(_oracle_slice, jobs)
    logp = res[0][0]
    leaves = np.concatenate([x[1] for x in res], axis=1)
    n = leaves.shape[1]
    if w.reward in ("neg_mse_mu", "neg_mse_target"):
        tgt = (inp.target if w.reward == "neg_mse_target" else inp.mu)[0][:n]
        r = np.array([rewards.neg_mse(leaves[q], tgt) for q in range(topo.leaves)])
    elif w.reward == "normal_plus_cos":
        r = np.array([float(inp.reward_draws[0][q]) + 0.1 * rewards.cosine(leaves[q], inp.target[0][:n]) for q in range(topo.leaves)])
    else:
        r = inp.reward_draws[0].astype(np.float64)
    rbar = credit.fuse_rewards(topo, r, logp, w.beta)
    credit.depth_advantages(topo, rbar, float(np.float32(w.eps)))
    credit.gradient_mask(topo, rbar.astype(np.float32), w.width_mode, w.width_k, inp.pruned_steps, w.ignore_last_step)
    dt = time.perf_counter() - t0
    frac = n_units / total_units
    if w.velocity == "linear":
        what = f"first {n_units * unit} of {w.D} elements"
    else:
        what = f"first {n_units} of {w.tokens} tokens"
    desc = f"1 of {w.n_trees} trees, {what}, all {topo.edges} node-steps; time x {1 / frac:.4g}"
    return dt, topo.edges / (dt / frac), desc


def _noop(_):
    return 0


ORACLE_SAMPLE = {   # (single-thread fraction, all-cores fraction) of one tree's latent row: about 10 s of CPU work each
    "toy": (1.0, 1.0), "image": (0.15, 1.0), "image_batch": (0.15, 1.0), "group": (0.05, 0.3), "video": (0.5, 1.0)}


def host_cores():
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def cpu_baseline(w, single=True):
    """The oracle on all host cores (one single-threaded process per core, at most 64) and on one core."""
    nproc = host_cores()
    workers = min(nproc, 64)
    f1, fn = ORACLE_SAMPLE.get(w.name, (0.02, 0.1))
    out = {"unit": UNIT, "kind": "oracle", "nproc": nproc}
    workers = max(1, min(workers, w.D // (4 if w.velocity == "linear" else w.channels)))
    dt_n, v_n, desc_n = oracle_pass(w, fn, workers)
    out.update({"value": r4(v_n), "cores": workers, "sample": desc_n, "sample_seconds": r4(dt_n)})
    if single:
        dt_1, v_1, desc_1 = oracle_pass(w, f1, 1)
        out["single_thread"] = {"value": r4(v_1), "cores": 1, "sample": desc_1, "sample_seconds": r4(dt_1)}
    return out


def run_reference(args, w):
    """The oracle arm: rank 0 alone computes and prints; the other ranks of a multi-rank launch only meet the barrier."""
    grp = RankGroup("gloo")
    if grp.rank == 0:
        vals, secs, base = [], [], None
        for k in range(args.warmup + args.steps):
            base = cpu_baseline(w, single=(k == args.warmup + args.steps - 1))
            if k >= args.warmup:
                vals.append(base["value"])
                secs.append(base["sample_seconds"])
        value = float(np.mean(vals))
        base["value"] = r4(value)
    grp.barrier()
    t = grp.max(float(np.mean(secs)) if grp.rank == 0 else 0.0)
    if grp.rank == 0:
        line = {
            "impl": "reference", "metric": METRIC, "value": r4(value), "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": r4(1e3 * w.n_trees * w.node_steps / value), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "description": w.description, "n_trees": w.n_trees,
                       "note": "CPU oracle on host cores (all cores, one process per core); ms_per_step is the full batch "
                               "extrapolated from the sample; sample_seconds is what one timed step took"},
            "cpu_baseline": base,
            "e2e": {"value": r4(value), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0, "sample_seconds_max_over_ranks": r4(t),
        }
        print(json.dumps(line))
    grp.close()


# ------------------------------------------------------------------------------------------------ per-kernel timing
def kernel_rooflines(s, w, peaks, flush_buf, reps):
    """Times every launch group of `reps` passes with in-stream events and returns (roofline of the dominant kernel,
    roofline of the step kernel, ms per pass by kernel).  An interval between two events holds one launch and the gap
    the event itself inserts (it also keeps the next launch's ramp from overlapping this launch's tail), so on
    workloads made of launches of a few microseconds the intervals add up to more than the un-instrumented pass."""
    import torch
    from paper_2509_06040_b200 import binding as B
    t_step, t_mlp = np.zeros(w.T), np.zeros(w.T)
    t_root, t_tail = 0.0, np.zeros(3)          # tail: leaf rewards, fusion + advantages, pruning masks

    def evs(n):
        return [torch.cuda.Event(enable_timing=True) for _ in range(n)]

    for rep in range(reps):
        if flush_buf is not None:
            flush_buf.fill_(1.0)
        e_init, e_tail, e_red = evs(2), evs(2), evs(2)
        e_lvl = [evs(3) for _ in range(w.T)]
        e_init[0].record()
        s.init(seed=w.seed + 3000 + rep)
        e_init[1].record()
        for i in range(w.T):
            e_lvl[i][0].record()
            if w.velocity == "mlp":
                B.velocity_mlp(s.tree, s.packed, w.hidden, s.v)
            e_lvl[i][1].record()
            B.tree_step(s.tree, 1 if i in w.splits else 0, s.v if w.velocity == "mlp" else None)
            e_lvl[i][2].record()
        e_tail[0].record()
        s.rewards()
        e_red[0].record()
        s.fuse_advantage()
        e_red[1].record()
        s.prune()
        e_tail[1].record()
        torch.cuda.synchronize()
        t_root += e_init[0].elapsed_time(e_init[1])
        t_tail += np.array([e_tail[0].elapsed_time(e_red[0]), e_red[0].elapsed_time(e_red[1]), e_red[1].elapsed_time(e_tail[1])])
        for i in range(w.T):
            t_mlp[i] += e_lvl[i][0].elapsed_time(e_lvl[i][1]) if w.velocity == "mlp" else 0.0
            t_step[i] += e_lvl[i][1].elapsed_time(e_lvl[i][2])
    t_step /= reps
    t_mlp /= reps
    t_root /= reps
    t_tail /= reps
    sb = np.array(step_bytes_per_launch(w, w.n_trees), dtype=np.float64)
    hbm_peak = float(peaks["hbm_gbs"])
    widest = int(np.argmax(sb))
    # launches that move more than the L2 holds are HBM launches whatever the previous launch left behind; the figure
    # the roofline reports is bytes over time of exactly those
    big = sb > 1.5 * L2_BYTES
    if big.any():
        gbs = float(sb[big].sum() / (t_step[big].sum() * 1e-3) / 1e9)
        basis = f"{int(big.sum())} of {w.T} launches, each > 1.5x L2"
    else:
        gbs = float(sb[widest] / (t_step[widest] * 1e-3) / 1e9)
        basis = "widest launch (all fit the L2)"
    roof_step = {"bound": "hbm", "kernel": "step_kernel", "achieved": r4(gbs), "peak": hbm_peak, "unit": "GB/s",
                 "frac": r4(gbs / hbm_peak), "frac_of_nominal_8TBs": r4(gbs / NOMINAL_HBM_GBS), "peak_source": peaks["_source"],
                 "basis": basis, "launches_per_pass": w.T, "ms_per_pass": r4(t_step.sum()),
                 "all_launches_gbs": r4(sb.sum() / (t_step.sum() * 1e-3) / 1e9),
                 "widest_launch": {"step": widest, "ms": r4(t_step[widest]), "gbs": r4(sb[widest] / (t_step[widest] * 1e-3) / 1e9)},
                 "traffic": r4(ncu_traffic("step_kernel_" + w.velocity, float(sum(c * w.D for c in step_children(w))) / w.T))}
    if w.velocity == "linear":
        # With the closed-form velocity the T step launches follow one another with nothing in between.  Between one pair
        # of events a launch's ramp overlaps its predecessor's tail and the level just written is still in the L2 when the
        # next launch reads it: bytes over this time is an algorithmic rate with L2 help, not HBM throughput.
        tot = 0.0
        for rep in range(reps):
            if flush_buf is not None:
                flush_buf.fill_(1.0)
            s.init(seed=w.seed + 4000 + rep)
            g0, g1 = evs(2)
            g0.record()
            for i in range(w.T - 1):      # the last step also enqueues the log-prob flush kernel: timed per launch above
                B.tree_step(s.tree, 1 if i in w.splits else 0, None)
            g1.record()
            B.tree_step(s.tree, 1 if (w.T - 1) in w.splits else 0, None)
            torch.cuda.synchronize()
            tot += g0.elapsed_time(g1)
        ms_group = tot / reps
        roof_step["algorithmic_gbs_l2_assisted"] = {"gbs": r4(sb[:-1].sum() / (ms_group * 1e-3) / 1e9), "ms": r4(ms_group),
                                                    "launches": w.T - 1}
    reward_bytes = 0.0 if w.reward == "mixture" else float(w.n_trees * (w.leaves + 1) * 4 * w.D)   # leaf rows once, target once per tree
    parts = {"mlp": t_mlp.sum(), "step": t_step.sum(), "root": t_root, "leaf_reward": t_tail[0], "fuse_advantage": t_tail[1],
             "prune": t_tail[2]}
    breakdown = {k: r4(v) for k, v in parts.items()}
    breakdown["sum"] = r4(sum(parts.values()))
    breakdown["leaf_reward_gbs"] = r4(reward_bytes / (t_tail[0] * 1e-3) / 1e9) if reward_bytes and t_tail[0] > 0 else None
    roof = roof_step
    if w.velocity == "mlp" and t_mlp.sum() > t_step.sum():
        fl = np.array(mlp_flops_per_launch(w, w.n_trees), dtype=np.float64)
        tf = fl.sum() / (t_mlp.sum() * 1e-3) / 1e12
        # a launch timed alone runs at burst clocks; inside a pass of many milliseconds the GPU sits at its power cap,
        # where the measured peak is the sustained one
        sustained = t_mlp.sum() >= 5.0 and "bf16_tflops_sustained" in peaks
        peak_tf = float(peaks["bf16_tflops_sustained"] if sustained else peaks["bf16_tflops"])
        wide = int(np.argmax(fl))
        roof = {"bound": "tensor", "kernel": "mlp_velocity_kernel", "achieved": r4(tf), "peak": peak_tf, "unit": "TFLOP/s",
                "frac": r4(tf / peak_tf), "peak_source": peaks["_source"],
                "peak_kind": "sustained" if sustained else "burst", "frac_of_burst_peak": r4(tf / float(peaks["bf16_tflops"])),
                "launches_per_pass": w.T, "ms_per_pass": r4(t_mlp.sum()),
                "widest_launch": {"step": wide, "tokens": int(fl[wide] / (4 * w.channels * w.hidden)), "ms": r4(t_mlp[wide]),
                                  "tflops": r4(fl[wide] / (t_mlp[wide] * 1e-3) / 1e12)},
                "traffic": r4(ncu_traffic("mlp_velocity_kernel", float(w.n_trees * w.model_evals * w.tokens) / w.T))}
    return roof, roof_step, breakdown


def fused_rollout_line(w, device, peaks, reps):
    """The same pass with all T steps in one launch (closed-form velocity): whole-pass throughput, and the rollout
    kernel alone against the bytes it must move (every node written once, root and target mean read once)."""
    import torch
    from paper_2509_06040_b200.session import TreeSession
    from paper_2509_06040_b200 import binding as B
    s = TreeSession(w, device=device, fused_rollout=True)
    s.upload_inputs(make_inputs(w))
    for k in range(2):
        s.run_all(seed=w.seed + k)
    torch.cuda.synchronize()
    a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a0.record()
    for k in range(reps):
        s.run_all(seed=w.seed + 100 + k)
    a1.record()
    torch.cuda.synchronize()
    ms = a0.elapsed_time(a1) / reps
    flags = [1 if i in w.splits else 0 for i in range(w.T)]
    t_k = 0.0
    for k in range(reps):
        s.init(seed=w.seed + 200 + k)
        b0, b1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        b0.record()
        B.tree_rollout_fused(s.tree, flags)
        b1.record()
        torch.cuda.synchronize()
        t_k += b0.elapsed_time(b1)
    t_k /= reps
    B.tree_sync_status(s.tree)
    nbytes = w.n_trees * (w.node_steps + 2) * 4.0 * w.D
    gbs = nbytes / (t_k * 1e-3) / 1e9
    out = {"value": r4(w.n_trees * w.node_steps / (ms * 1e-3)), "ms_per_step": r4(ms),
           "roofline": {"bound": "hbm", "kernel": "rollout_fused_kernel", "achieved": r4(gbs), "peak": float(peaks["hbm_gbs"]),
                        "unit": "GB/s", "frac": r4(gbs / float(peaks["hbm_gbs"])), "frac_of_nominal_8TBs": r4(gbs / NOMINAL_HBM_GBS),
                        "bytes_per_launch": nbytes, "ms_per_launch": r4(t_k),
                        "traffic": r4(ncu_traffic("rollout_fused_kernel", float(w.n_trees * w.node_steps * w.D)))}}
    del s
    torch.cuda.empty_cache()
    return out


def savings_line(w, s_tree, device, reps):
    """The tree against an equal-leaf-count batch of independent sequential rollouts through the same kernels
    (K = 1, no split, n_trees x leaves trees of T steps): model evaluations and measured rollout time."""
    import torch
    from paper_2509_06040_b200.session import TreeSession

    def rollout_ms(sess, ww):
        for k in range(2):
            sess.rollout(seed=ww.seed + 5000 + k)
        torch.cuda.synchronize()
        a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a0.record()
        for k in range(reps):
            sess.rollout(seed=ww.seed + 5100 + k)
        a1.record()
        torch.cuda.synchronize()
        return a0.elapsed_time(a1) / reps

    t_tree = rollout_ms(s_tree, w)
    wseq = w.scaled(name=w.name + "_sequential", n_trees=w.n_trees * w.leaves, K=1, splits=())
    seq = TreeSession(wseq, device=device)
    seq.upload_inputs(make_inputs(wseq))
    t_seq = rollout_ms(seq, wseq)
    del seq
    torch.cuda.empty_cache()
    return {"final_samples": w.n_trees * w.leaves, "model_evals_tree": w.n_trees * w.model_evals,
            "model_evals_sequential": w.n_trees * w.leaves * w.T, "model_evals_ratio": r4((w.leaves * w.T) / w.model_evals),
            "rollout_ms_tree": r4(t_tree), "rollout_ms_sequential": r4(t_seq), "rollout_time_ratio": r4(t_seq / t_tree)}


def brief_workload(name, device, peaks):
    """Another named workload, briefly (single GPU): whole-pass throughput and the two kernels' rooflines, compact."""
    import torch
    from paper_2509_06040_b200.session import TreeSession
    w2 = CONFIGS[name]
    s2 = TreeSession(w2, device=device)
    s2.upload_inputs(make_inputs(w2))
    pool_bytes = s2.latents.numel() * 4
    flush_buf = torch.empty(3 * L2_BYTES // 4, dtype=torch.float32, device=s2.device) if pool_bytes <= 2 * L2_BYTES else None
    for k in range(3):
        s2.run_all(seed=w2.seed + k)
    torch.cuda.synchronize()
    n2 = 10
    tot = 0.0
    for k in range(n2):
        if flush_buf is not None:
            flush_buf.fill_(float(k))
        a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a0.record()
        s2.run_all(seed=w2.seed + 100 + k)
        a1.record()
        torch.cuda.synchronize()
        tot += a0.elapsed_time(a1)
    ms = tot / n2
    r2, rs2, bd2 = kernel_rooflines(s2, w2, peaks, flush_buf, 3)

    def compact(r):
        keep = ("kernel", "achieved", "peak", "unit", "frac", "frac_of_nominal_8TBs", "peak_kind", "basis")
        out = {k: r[k] for k in keep if k in r}
        if "widest_launch" in r:
            out["widest_launch"] = {k: r["widest_launch"][k] for k in ("ms", "gbs", "tflops") if k in r["widest_launch"]}
        if "algorithmic_gbs_l2_assisted" in r:
            out["algorithmic_gbs_l2_assisted"] = r["algorithmic_gbs_l2_assisted"]["gbs"]
        return out

    out = {"value": r4(w2.n_trees * w2.node_steps / (ms * 1e-3)), "ms_per_step": r4(ms), "roofline": compact(r2),
           "kernel_ms_sum": bd2["sum"]}
    if r2 is not rs2:
        out["roofline_step"] = compact(rs2)
    del s2, flush_buf
    torch.cuda.empty_cache()
    if w2.velocity == "linear":
        fr = fused_rollout_line(w2, device, peaks, n2)
        out["one_launch_rollout"] = {"value": fr["value"], "ms_per_step": fr["ms_per_step"],
                                     "gbs": fr["roofline"]["achieved"], "frac": fr["roofline"]["frac"]}
    return out


# ------------------------------------------------------------------------------------------------ GPU arm
def run_ours(args, w):
    import torch
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    grp = RankGroup("nccl", device)
    world, rank = grp.world, grp.rank
    import __graft_entry__
    if rank == 0:
        __graft_entry__.build()
    grp.barrier()
    from paper_2509_06040_b200.session import TreeSession
    from paper_2509_06040_b200 import binding as B

    # weak scaling: every rank holds the workload's n_trees trees, with its own global tree indices
    base = rank * w.n_trees
    inp = make_inputs(w, tree_base=base)
    s = TreeSession(w, tree_id_base=base, device=f"cuda:{local}", fused_rollout=args.fused_rollout)
    s.upload_inputs(inp)
    pool_bytes = s.latents.numel() * 4
    flush = pool_bytes <= 2 * L2_BYTES
    flush_buf = torch.empty(3 * L2_BYTES // 4, dtype=torch.float32, device=s.device) if flush else None

    def sync_all():
        grp.barrier()
        torch.cuda.synchronize()

    for k in range(args.warmup):
        s.run_all(seed=w.seed + k)
    torch.cuda.synchronize()
    B.tree_sync_status(s.tree)

    # ---- timed region: K passes, device-timed with CUDA events on the launching stream
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    sampler = ClockSampler(local) if rank == 0 else None
    sync_all()
    for k in range(args.steps):
        if flush:
            flush_buf.fill_(float(k))
        ev[k][0].record()
        s.run_all(seed=w.seed + 1000 + k)
        ev[k][1].record()
    sync_all()
    clocks = sampler.stop() if sampler else None
    total_ms = grp.max(sum(a.elapsed_time(b) for a, b in ev))
    node_steps_per_pass = world * w.n_trees * w.node_steps
    value = node_steps_per_pass * args.steps / (total_ms * 1e-3)

    # ---- end to end through the C ABI with host buffers: H2D of the step's inputs (pinned), D2H of its results
    host_in = {}
    for name in ("mu", "target", "reward_draws"):
        a = getattr(inp, name)
        if a is not None:
            host_in[name] = torch.from_numpy(a).pin_memory()
    host_out = {n: torch.empty_like(getattr(s, n), device="cpu").pin_memory() for n in ("adv", "mask", "logp", "leaf_r")}
    h2d = sum(x.numel() * x.element_size() for x in host_in.values())
    d2h = sum(x.numel() * x.element_size() for x in host_out.values())

    def e2e_pass(k):
        for name, h in host_in.items():
            getattr(s, name).copy_(h, non_blocking=True)
        s.run_all(seed=w.seed + 2000 + k)
        for name, h in host_out.items():
            h.copy_(getattr(s, name), non_blocking=True)

    for k in range(2):
        e2e_pass(k)
    sync_all()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    n_e2e = max(3, args.steps // 2)
    e2e_ms = 0.0
    for k in range(n_e2e):
        if flush:
            flush_buf.fill_(float(k))
        e0.record()
        e2e_pass(k)
        e1.record()
        e1.synchronize()
        e2e_ms += e0.elapsed_time(e1)
    e2e_serial = node_steps_per_pass * n_e2e / (grp.max(e2e_ms) * 1e-3)

    # The same passes as a stream of work: the inputs of pass k+1 cross PCIe on a second stream (into one of two staging
    # buffers) while pass k computes; every pass still takes its inputs from pinned host memory and returns its results.
    copy_stream = torch.cuda.Stream(device=s.device)
    stage = [{n: torch.empty_like(getattr(s, n)) for n in host_in} for _ in range(2)]
    copied = [torch.cuda.Event() for _ in range(2)]
    consumed = [torch.cuda.Event() for _ in range(2)]

    def issue_copy(k):
        b = k & 1
        with torch.cuda.stream(copy_stream):
            if k >= 2:
                copy_stream.wait_event(consumed[b])
            for name, h in host_in.items():
                stage[b][name].copy_(h, non_blocking=True)
            copied[b].record(copy_stream)

    def piped_pass(k):
        b = k & 1
        cur = torch.cuda.current_stream()
        cur.wait_event(copied[b])
        for name in host_in:
            getattr(s, name).copy_(stage[b][name])
        consumed[b].record(cur)
        s.run_all(seed=w.seed + 2500 + k)
        for name, h in host_out.items():
            h.copy_(getattr(s, name), non_blocking=True)

    sync_all()
    if flush:
        flush_buf.fill_(1.0)
    e0.record()
    issue_copy(0)
    for k in range(n_e2e):
        if k + 1 < n_e2e:
            issue_copy(k + 1)
        piped_pass(k)
    e1.record()
    e1.synchronize()
    torch.cuda.synchronize()
    e2e_value = node_steps_per_pass * n_e2e / (grp.max(e0.elapsed_time(e1)) * 1e-3)

    # ---- per-kernel durations, measured live with events around each launch (rank 0)
    roof = roof_step = None
    breakdown = {}
    peaks = load_peaks()
    if rank == 0:
        if s.fused_rollout:
            roof = roof_step = fused_rollout_line(w, f"cuda:{local}", peaks, max(3, min(10, args.steps)))["roofline"]
        else:
            roof, roof_step, breakdown = kernel_rooflines(s, w, peaks, flush_buf, max(3, min(10, args.steps)))
            breakdown["pass"] = r4(total_ms / args.steps)
            breakdown["note"] = ("one event interval per launch; each holds the event's own gap, so the sum exceeds the pass "
                                 "where launches take microseconds" if breakdown["sum"] > 1.1 * breakdown["pass"]
                                 else "one event interval per launch")

    # ---- the tree against independent sequential rollouts with as many final samples (rank 0, single GPU)
    savings = None
    if rank == 0 and world == 1 and not args.no_also:
        savings = savings_line(w, s, f"cuda:{local}", max(3, min(10, args.steps)))
    launches = s.kernel_launches_per_pass() * args.steps
    dtype = "f32" if w.velocity == "linear" else "f32 (step) + bf16/f32-accumulate (MLP velocity)"
    rollout_kind = "one launch" if s.fused_rollout else "one tree_step per depth"
    del s, stage, flush_buf
    torch.cuda.empty_cache()

    # ---- the other image- and video-shaped workloads, briefly (rank 0, single GPU): same path, same timing method
    also = {}
    if rank == 0 and world == 1 and not args.no_also:
        for name in ("image_batch", "video", "image", "group"):
            if name != w.name:
                also[name] = brief_workload(name, f"cuda:{local}", peaks)

    # ---- CPU oracle on a bounded sample (rank 0, single GPU runs only)
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu = cpu_baseline(w)

    if rank == 0:
        line = {
            "metric": METRIC, "value": r4(value), "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": r4(total_ms / args.steps), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": dtype, "data": "synthetic",
            "config": {"workload": w.name, "n_trees_per_gpu": w.n_trees, "tokens": w.tokens, "channels": w.channels, "T": w.T,
                       "splits": list(w.splits), "velocity": w.velocity, "node_steps_per_tree": w.node_steps,
                       "model_evals_per_tree": w.model_evals, "latent_pool_bytes": pool_bytes,
                       "l2": "flushed between steps" if flush else "pool larger than L2",
                       "rollout": rollout_kind, "parallelism": f"dp{world} over trees, no collective"},
            "roofline": roof, "cpu_baseline": cpu,
            "e2e": {"value": r4(e2e_value), "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "mode": "next pass's inputs copied under this pass", "one_pass_at_a_time": r4(e2e_serial)},
            "gpu_launches": launches, "clocks": clocks, "kernel_ms_per_pass": breakdown, "savings": savings, "also": also,
        }
        if roof is not roof_step:
            line["roofline_step"] = roof_step
        print(json.dumps(line))
    grp.close()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="group", choices=list(CONFIGS),
                    help="default: group, the largest single-GPU configuration (8 trees x 765 nodes x 4096 x 64, MLP velocity)")
    ap.add_argument("--fused-rollout", action="store_true",
                    help="closed-form-velocity workloads: all T steps in one launch (tree_rollout_fused)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-also", action="store_true", help="skip the brief runs of the other workloads and the savings run")
    args = ap.parse_args()
    if args.gpus > 1 and "RANK" not in os.environ:
        sys.exit(spawn_ranks(args.gpus, sys.argv[1:]))
    w = CONFIGS[args.workload]
    if args.impl == "reference":
        args.steps = min(args.steps, 3)      # each step is seconds of CPU work on a bounded sample
        args.warmup = min(args.warmup, 1)
        run_reference(args, w)
    else:
        args.warmup = max(args.warmup, 3)
        run_ours(args, w)


if __name__ == "__main__":
    main()
