"""`bench.py --gpus N` starts its N ranks itself (one process per GPU under torch.distributed.run).  Here the launch
path runs on CPU with the oracle arm as the compute: two ranks come up over gloo, meet the barrier, reduce the measured
time with MAX over ranks, and rank 0 alone prints the one JSON line, with n_gpus = 2 and the oracle's single-thread and
all-cores figures."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(extra):
    env = dict(os.environ)
    for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT"):
        env.pop(k, None)
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "toy",
                          "--steps", "1", "--warmup", "0"] + extra, capture_output=True, text=True, timeout=600, env=env, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, out.stdout
    return json.loads(lines[0])


def test_two_ranks_are_spawned_and_rank_zero_prints_one_line():
    line = _run(["--gpus", "2"])
    assert line["impl"] == "reference" and line["n_gpus"] == 2
    assert line["unit"] == "node-steps/s" and line["value"] > 0 and line["higher_is_better"] is True
    base = line["cpu_baseline"]
    assert base["kind"] == "oracle" and base["cores"] >= 1 and base["nproc"] >= base["cores"] >= 1
    assert base["single_thread"]["cores"] == 1 and base["single_thread"]["value"] > 0
    assert line["e2e"] == {"value": line["value"], "unit": line["unit"], "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert line["sample_seconds_max_over_ranks"] == base["sample_seconds"]      # MAX over ranks: rank 1 contributes 0


def test_rank_group_without_a_launcher_is_a_single_rank():
    sys.path.insert(0, ROOT)
    import bench
    saved = {k: os.environ.pop(k, None) for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    try:
        g = bench.RankGroup("gloo")
        assert (g.world, g.rank) == (1, 0)
        g.barrier()
        assert g.max(3.5) == 3.5
        g.close()
    finally:
        for k, v in saved.items():
            if v is not None:
                os.environ[k] = v
