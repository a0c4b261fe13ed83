#!/usr/bin/env python
"""Benchmark of the BranchGRPO tree hot path: tree node-steps/s and achieved HBM bandwidth.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

One "step" is one pass of the whole path over one batch of synthetic trees: root init, T x
[velocity, fused tree step], leaf rewards, reward fusion + depth-wise advantages, pruning masks.
A node-step is one edge of a tree (one child latent with its log-prob).  With N > 1 (launched by
torch.distributed.run) every rank runs its own shard of trees - the path has no exchange step -
and the reported value is all ranks' node-steps over the slowest rank's time (weak scaling).

`--impl reference` times the CPU oracle (oracle/), as it stands, on a bounded sample of the same
workload on this machine's host cores; it is a deliberately slow program and a reported baseline.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import re
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

# DRAM traffic of the dominant kernel from one ncu capture (dram__bytes_read.sum + dram__bytes_write.sum), see
# profiles/.  Each entry is the captured launch's bytes and the units (elements / tokens) it processed; the figure
# reported per launch is bytes-per-unit times the units of an average launch of the timed workload (traffic grows in
# proportion to the units).  It is reported only while the kernel's sources still hash to what was captured.
NCU_TRAFFIC = {
    "step_kernel": {"workload": "video", "bytes": 75.599616e6 + 12.611840e6, "units": 8 * 2096640,
                    "sources": ("tree_step.cu", "philox.cuh"), "shape": "kStep", "source_hash": "0f5299a50f5b"},
    "mlp_velocity_kernel": {"workload": "image_batch", "bytes": 266.295808e6 + 214.387712e6, "units": 1036800,
                            "sources": ("mlp_velocity.cu",), "shape": "kMlp", "source_hash": "2141aa3f7a6b"},
    "rollout_fused_kernel": {"workload": "video", "bytes": 16.817152e6 + 866.026752e6, "units": 110 * 2096640,
                             "sources": ("tree_fused.cu", "philox.cuh"), "shape": "kFused", "source_hash": "b6671b3e66cb"},
}


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


# ------------------------------------------------------------------------------------------------ algorithmic bytes
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
                                       "--format=csv,noheader,nounits", "-lms", "100"], stdout=self.f, stderr=subprocess.DEVNULL)
        except OSError:
            self.p = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.p is None:
            return out
        time.sleep(0.15)
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
        sm = [float(r[0]) for r in rows]
        out["sm_mhz"] = float(np.median(sm))
        out["sm_max_mhz"] = float(rows[0][1])
        out["power_w_max"] = max(float(r[2]) for r in rows)
        out["samples"] = len(rows)
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for k, nm in enumerate(names):
            if any("Active" == r[4 + k].strip() for r in rows):
                out["reasons"].append(nm)
        return out


# ------------------------------------------------------------------------------------------------ oracle timing
def oracle_pass(w, inp, sample):
    """One pass of the oracle over a bounded sample of workload `w`.  Returns (seconds, node-steps of the
    FULL per-GPU workload that this time corresponds to after linear scaling, description, threads)."""
    from oracle import credit, mlp, rewards, sde
    from oracle import tree as otree
    topo = otree.build_topology(w.T, w.K, w.splits)
    grid = w.t_grid().astype(np.float64)
    sig, s0 = float(np.float32(w.sigma)), float(np.float32(w.s0))
    t0 = time.perf_counter()
    if w.velocity == "linear":
        n_elem = max(4, (int(w.D * sample) // 4) * 4)
        mu = inp.mu[0][:n_elem].astype(np.float64)
        lat, logp = sde.rollout(topo, n_elem, grid, sig, w.branch_corr_s, w.seed,
                                lambda z, i, p: sde.linear_velocity(z.astype(np.float64), float(grid[i]), mu, s0))
        tgt = (inp.target if inp.target is not None else inp.mu)[0][:n_elem]
        r = np.array([rewards.neg_mse(lat[l], tgt) for l in topo.leaf_ids()])
        frac = n_elem / w.D
        desc = f"1 of {w.n_trees} trees, first {n_elem} of {w.D} elements per node, all {topo.edges} node-steps; time scaled by D/sample"
        threads = 1
    else:
        n_tok = max(1, int(w.tokens * sample))
        D_s = n_tok * w.channels
        vel = lambda z, i, p: mlp.mlp_velocity(z.reshape(n_tok, w.channels), inp.W1, inp.W2).reshape(-1)
        lat, logp = sde.rollout(topo, D_s, grid, sig, w.branch_corr_s, w.seed, vel)
        if inp.target is not None:
            r = np.array([float(inp.reward_draws[0][q]) + 0.1 * rewards.cosine(lat[l], inp.target[0][:D_s])
                          for q, l in enumerate(topo.leaf_ids())])
        else:
            r = inp.reward_draws[0].astype(np.float64)
        frac = n_tok / w.tokens
        desc = f"1 of {w.n_trees} trees, first {n_tok} of {w.tokens} tokens per node, all {topo.edges} node-steps; time scaled by tokens/sample"
        threads = _blas_threads()
    rbar = credit.fuse_rewards(topo, r, logp, w.beta)
    credit.depth_advantages(topo, rbar, float(np.float32(w.eps)))
    credit.gradient_mask(topo, rbar.astype(np.float32), w.width_mode, w.width_k, inp.pruned_steps, w.ignore_last_step)
    dt = time.perf_counter() - t0
    full_seconds_one_tree = dt / frac
    return dt, topo.edges / full_seconds_one_tree, desc, threads


def _blas_threads():
    try:
        from threadpoolctl import threadpool_info
        return max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        return os.cpu_count() or 1


def oracle_sample_fraction(w):
    return {"toy": 1.0, "image": 0.4, "image_batch": 0.4, "group": 0.05, "video": 1.0}.get(w.name, 0.05)


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    inp = make_inputs(w.scaled(n_trees=1))
    frac = oracle_sample_fraction(w)
    for _ in range(args.warmup):
        oracle_pass(w, inp, frac / 8)
    vals, secs = [], []
    for _ in range(args.steps):
        dt, v, desc, threads = oracle_pass(w, inp, frac)
        vals.append(v)
        secs.append(dt)
    value = float(np.mean(vals))
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * w.n_trees * w.node_steps / value, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "description": w.description, "n_trees": w.n_trees,
                   "note": "CPU oracle on host cores; ms_per_step is the full batch extrapolated from the sample"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc,
                         "sample_seconds": float(np.mean(secs))},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def kernel_rooflines(s, w, peaks, flush_buf, reps):
    """Times every velocity and step launch of `reps` passes with in-stream events and returns
    (roofline of the dominant kernel, roofline of the step kernel, ms per pass by kernel group)."""
    import torch
    from paper_2509_06040_b200 import binding as B
    t_step = np.zeros(w.T)
    t_mlp = np.zeros(w.T)
    t_other = 0.0
    t_tail = np.zeros(3)          # leaf rewards, fusion + advantages, pruning masks

    def evs(n):
        return [torch.cuda.Event(enable_timing=True) for _ in range(n)]

    for rep in range(reps):
        # events are recorded back to back on the launching stream and read after one final synchronize,
        # so an interval holds one launch (plus its in-stream launch gap), never a host round trip
        if flush_buf is not None:
            flush_buf.fill_(1.0)
        e_init, e_tail = evs(2), evs(2)
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
        e_red = evs(2)
        e_tail[0].record()
        s.rewards()
        e_red[0].record()
        s.fuse_advantage()
        e_red[1].record()
        s.prune()
        e_tail[1].record()
        torch.cuda.synchronize()
        t_other += e_init[0].elapsed_time(e_init[1]) + e_tail[0].elapsed_time(e_tail[1])
        t_tail += np.array([e_tail[0].elapsed_time(e_red[0]), e_red[0].elapsed_time(e_red[1]), e_red[1].elapsed_time(e_tail[1])])
        for i in range(w.T):
            t_mlp[i] += e_lvl[i][0].elapsed_time(e_lvl[i][1]) if w.velocity == "mlp" else 0.0
            t_step[i] += e_lvl[i][1].elapsed_time(e_lvl[i][2])
    t_step /= reps
    t_mlp /= reps
    t_other /= reps
    t_tail /= reps
    sb = np.array(step_bytes_per_launch(w, w.n_trees), dtype=np.float64)
    step_gbs_events = sb.sum() / (t_step.sum() * 1e-3) / 1e9
    step_ms_group = None
    if w.velocity == "linear":
        # With the closed-form velocity the T step launches follow one another with nothing in between: one pair of events
        # around the group gives their average duration without the gap that an event between two launches costs.
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
        step_ms_group = tot / reps
    if step_ms_group is not None:
        step_gbs = sb[:-1].sum() / (step_ms_group * 1e-3) / 1e9
    else:
        step_gbs = step_gbs_events
    widest = int(np.argmax(sb))
    hbm_peak = float(peaks["hbm_gbs"])
    roof_step = {"bound": "hbm", "kernel": "step_kernel", "achieved": step_gbs, "peak": hbm_peak, "unit": "GB/s",
                 "frac": step_gbs / hbm_peak, "frac_of_nominal_8TBs": step_gbs / NOMINAL_HBM_GBS,
                 "peak_source": peaks["_source"], "launches_per_pass": w.T,
                 "bytes_per_pass": float(sb.sum()), "ms_per_pass": float(t_step.sum()),
                 "timing": ("steps 0..T-2 back to back between one pair of events (%.4f ms for %.0f bytes)" % (step_ms_group, sb[:-1].sum()))
                           if step_ms_group is not None else "one pair of events per launch",
                 "gbs_with_an_event_between_launches": step_gbs_events,
                 "widest_launch": {"step": widest, "bytes": float(sb[widest]), "ms": float(t_step[widest]),
                                   "gbs": float(sb[widest] / (t_step[widest] * 1e-3) / 1e9)},
                 "traffic": ncu_traffic("step_kernel", float(sum(c * w.D for c in step_children(w))) / w.T)}
    reward_bytes = 0.0 if w.reward == "mixture" else float(w.n_trees * (w.leaves + 1) * 4 * w.D)   # leaf rows once, target once per tree
    breakdown = {"step_ms": float(t_step.sum()), "mlp_ms": float(t_mlp.sum()), "other_ms": float(t_other),
                 "leaf_reward_ms": float(t_tail[0]), "fuse_advantage_ms": float(t_tail[1]), "prune_ms": float(t_tail[2]),
                 "leaf_reward_gbs": (reward_bytes / (t_tail[0] * 1e-3) / 1e9) if reward_bytes and t_tail[0] > 0 else None,
                 "note": "intervals between in-stream events: each holds one launch and its launch gap; the reduction "
                         "kernels handle a few hundred scalars per tree and are latency-bound"}
    roof = roof_step
    if w.velocity == "mlp" and t_mlp.sum() > t_step.sum():
        fl = np.array(mlp_flops_per_launch(w, w.n_trees), dtype=np.float64)
        tf = fl.sum() / (t_mlp.sum() * 1e-3) / 1e12
        # a launch timed alone runs at burst clocks; inside a pass of many milliseconds the GPU sits at its power cap,
        # where the measured peak is the sustained one
        sustained = t_mlp.sum() >= 5.0 and "bf16_tflops_sustained" in peaks
        peak_tf = float(peaks["bf16_tflops_sustained"] if sustained else peaks["bf16_tflops"])
        # one hardware tanh per hidden activation: the XU pipe issues 16 per clock per SM
        sms = torch.cuda.get_device_properties(s.device).multi_processor_count
        xu_peak = 16.0 * sms * float(peaks.get("sm_max_mhz", 1965.0)) * 1e6
        tanh_rate = fl.sum() / (4.0 * w.channels) / (t_mlp.sum() * 1e-3)
        roof = {"bound": "tensor", "kernel": "mlp_velocity_kernel", "achieved": tf, "peak": peak_tf, "unit": "TFLOP/s",
                "frac": tf / peak_tf, "peak_source": peaks["_source"],
                "peak_kind": "sustained (%.1f ms of MLP launches per pass)" % t_mlp.sum() if sustained else "burst (short launches)",
                "frac_of_burst_peak": tf / float(peaks["bf16_tflops"]), "launches_per_pass": w.T,
                "flops_per_pass": float(fl.sum()), "ms_per_pass": float(t_mlp.sum()),
                "note": "a dense contraction, so reported against the tensor peak; the pipe that binds it is the XU "
                        "(one hardware tanh per hidden activation), see xu_bound",
                "xu_bound": {"bound": "alu", "unit": "Gtanh/s", "achieved": tanh_rate / 1e9, "peak": xu_peak / 1e9,
                             "frac": tanh_rate / xu_peak, "peak_source": "16 tanh/clk/SM x SMs x max SM clock"},
                "traffic": ncu_traffic("mlp_velocity_kernel", float(w.n_trees * w.model_evals * w.tokens) / w.T)}
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
    out = {"value": w.n_trees * w.node_steps / (ms * 1e-3), "unit": UNIT, "ms_per_step": ms, "steps": reps,
           "gpu_launches_per_pass": s.kernel_launches_per_pass(),
           "roofline": {"bound": "hbm", "kernel": "rollout_fused_kernel (+ its log-prob sums)", "achieved": gbs,
                        "peak": float(peaks["hbm_gbs"]), "unit": "GB/s", "frac": gbs / float(peaks["hbm_gbs"]),
                        "peak_source": peaks["_source"], "bytes_per_launch": nbytes, "ms_per_launch": t_k,
                        "traffic": ncu_traffic("rollout_fused_kernel", float(w.n_trees * w.node_steps * w.D)),
                        "note": "4 bytes per element and node-step (write only); the kernel is bound by instruction issue "
                                "(Philox + Box-Muller), like the step kernel on this workload"}}
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
    return {"leaves": w.n_trees * w.leaves, "model_evals_tree": w.n_trees * w.model_evals,
            "model_evals_sequential": w.n_trees * w.leaves * w.T,
            "model_evals_ratio": (w.leaves * w.T) / w.model_evals,
            "rollout_ms_tree": t_tree, "rollout_ms_sequential": t_seq, "rollout_time_ratio": t_seq / t_tree,
            "note": "sequential = the same number of final samples as independent T-step rollouts (K = 1) through the same kernels"}


# ------------------------------------------------------------------------------------------------ GPU arm
def run_ours(args, w):
    import torch
    import torch.distributed as dist
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    import __graft_entry__
    if rank == 0:
        __graft_entry__.build()
    if world > 1:
        dist.barrier()
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
        if world > 1:
            dist.barrier()
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
    total_ms = sum(a.elapsed_time(b) for a, b in ev)
    t = torch.tensor([total_ms], dtype=torch.float64, device=s.device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    total_ms = float(t.item())
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
    t = torch.tensor([e2e_ms], dtype=torch.float64, device=s.device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    e2e_serial = node_steps_per_pass * n_e2e / (float(t.item()) * 1e-3)

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
    t = torch.tensor([e0.elapsed_time(e1)], dtype=torch.float64, device=s.device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    e2e_value = node_steps_per_pass * n_e2e / (float(t.item()) * 1e-3)

    # ---- per-kernel durations, measured live with events around each launch (rank 0)
    roof = roof_step = None
    breakdown = {}
    if rank == 0:
        peaks = load_peaks()
        if s.fused_rollout:
            roof = roof_step = fused_rollout_line(w, f"cuda:{local}", peaks, max(3, min(10, args.steps)))["roofline"]
        else:
            roof, roof_step, breakdown = kernel_rooflines(s, w, peaks, flush_buf, max(3, min(10, args.steps)))

    # ---- the other image- and video-shaped workloads, briefly (rank 0, single GPU): same path, same timing method
    also = {}
    if rank == 0 and world == 1 and not args.no_also:
        for name in ("image_batch", "video"):
            if name == w.name:
                continue
            w2 = CONFIGS[name]
            s2 = TreeSession(w2, device=f"cuda:{local}")
            s2.upload_inputs(make_inputs(w2))
            for k in range(2):
                s2.run_all(seed=w2.seed + k)
            torch.cuda.synchronize()
            n2 = 10
            a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a0.record()
            for k in range(n2):
                s2.run_all(seed=w2.seed + 100 + k)
            a1.record()
            torch.cuda.synchronize()
            ms = a0.elapsed_time(a1) / n2
            r2, rs2, bd2 = kernel_rooflines(s2, w2, peaks, None, 3)
            also[name] = {"value": w2.n_trees * w2.node_steps / (ms * 1e-3), "unit": UNIT, "ms_per_step": ms, "steps": n2,
                          "l2": "latent pool larger than L2", "roofline": r2, "roofline_step": rs2, "kernel_ms_per_pass": bd2}
            del s2
            torch.cuda.empty_cache()
            if w2.velocity == "linear":
                also[name]["fused_rollout"] = fused_rollout_line(w2, f"cuda:{local}", peaks, n2)

    # ---- the tree against independent sequential rollouts with as many final samples (rank 0, single GPU)
    savings = None
    if rank == 0 and world == 1 and not args.no_also:
        savings = savings_line(w, s, f"cuda:{local}", max(3, min(10, args.steps)))

    # ---- CPU oracle on a bounded sample (rank 0, single GPU runs only)
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        inp1 = make_inputs(w.scaled(n_trees=1))
        dt, v, desc, threads = oracle_pass(w, inp1, oracle_sample_fraction(w))
        cpu = {"value": v, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc, "sample_seconds": dt}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32" if w.velocity == "linear" else "f32 (step) + bf16/f32-accumulate (MLP velocity)",
            "data": "synthetic",
            "config": {"workload": w.name, "description": w.description, "n_trees_per_gpu": w.n_trees,
                       "tokens": w.tokens, "channels": w.channels, "T": w.T, "K": w.K, "splits": list(w.splits),
                       "node_steps_per_tree": w.node_steps, "model_evals_per_tree": w.model_evals,
                       "model_evals_sequential": w.leaves * w.T, "latent_pool_bytes": pool_bytes,
                       "l2": "flushed between steps (pool fits in L2)" if flush else "latent pool larger than L2",
                       "rollout": "one launch (tree_rollout_fused)" if s.fused_rollout else "one tree_step launch per depth",
                       "parallelism": f"dp{world} over trees, no collective"},
            "roofline": roof, "cpu_baseline": cpu,
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "mode": "stream of passes: inputs of pass k+1 copied from pinned host memory on a second stream while "
                            "pass k computes; results of every pass copied back to pinned host memory",
                    "one_pass_at_a_time": e2e_serial},
            "gpu_launches": s.kernel_launches_per_pass() * args.steps,
            "clocks": clocks, "kernel_ms_per_pass": breakdown, "savings": savings, "also": also,
        }
        if roof is not roof_step:
            line["roofline_step"] = roof_step
        print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="image", choices=list(CONFIGS))
    ap.add_argument("--fused-rollout", action="store_true",
                    help="closed-form-velocity workloads: all T steps in one launch (tree_rollout_fused)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-also", action="store_true", help="skip the brief runs of the other image/video workloads")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    w = CONFIGS[args.workload]
    if args.impl == "reference":
        args.steps = min(args.steps, 3)      # each step is 10-20 s of CPU work on a bounded sample
        args.warmup = min(args.warmup, 1)
        run_reference(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
