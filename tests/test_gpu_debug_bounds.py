"""The build with device-side index checks (libbgrpo_debug.so, -DBGRPO_DEBUG_BOUNDS): every kernel tests the row,
chunk and element indices it derives against the extents of its launch, sets a status bit and skips the access on a
miss.  A child process that loads that build (BGRPO_DEBUG_BOUNDS=1) runs whole passes over the toy tree, the ragged
shapes, K = 3 and K = 4 trees, the MLP stage and the one-launch rollout and finds the status word clean after each; it
also makes one check fail on purpose (a kernel that touches no memory) and sees the failure reported.  The parity tests
of those shapes are then run once more against the debug build."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

SCRIPT = r'''
import math, sys
import numpy as np, torch
sys.path.insert(0, "tests")
from paper_2509_06040_b200 import binding as B
from paper_2509_06040_b200.session import TreeSession
from workloads import CONFIGS, Workload, make_inputs
from test_gpu_parity import RAGGED
assert B.DEBUG_BOUNDS and B.LIB_PATH.endswith("libbgrpo_debug.so")
B.debug_bounds(None)                                     # OK only in the debug build
cases = [CONFIGS["toy"]]
for name, n_trees, tokens, channels, T, K, splits, sigma, s_corr, base, extra in RAGGED:
    cases.append(Workload(name=name, n_trees=n_trees, tokens=tokens, channels=channels, T=T, K=K, splits=splits, sigma=sigma,
                          velocity="linear", reward="neg_mse_mu", branch_corr_s=s_corr, width_mode=B.WIDTH_EXTREME_B, width_k=2))
cases.append(Workload(name="mlp_k3", n_trees=3, tokens=171, channels=64, T=4, K=3, splits=(0, 2), sigma=0.3, velocity="mlp",
                      reward="normal_plus_cos", hidden=256, width_mode=B.WIDTH_PER_SPLIT_TOPK, width_k=1, n_pruned_depths=2))
for w in cases:
    for fused in ((False, True) if w.velocity == "linear" else (False,)):
        s = TreeSession(w, nodes_cap=w.nodes + 3, fused_rollout=fused)
        s.upload_inputs(make_inputs(w))
        for seed in (1, 2):
            s.run_all(seed=seed)
        out = torch.zeros_like(s.logp)
        if w.velocity == "linear":
            B.tree_logprob(s.tree, -1, None, out)
        else:
            B.tree_logprob(s.tree, w.T - 1, s.v, out)
        B.tree_fusion_ess(s.tree, 1.0, 1.0, out)
        J = torch.zeros(w.n_trees, device="cuda")
        B.tree_grpo_objective(s.tree, s.logp, None, 1.0, 0.2, out, J)
        torch.cuda.synchronize()
        B.tree_sync_status(s.tree)                       # raises if any index check failed
        assert torch.isfinite(s.latents[:, :w.nodes]).all()
# the reporting path: one check fails on purpose, nothing is accessed
B.debug_bounds(s.tree, trip=True)
try:
    B.tree_sync_status(s.tree)
    raise SystemExit("the tripped check was not reported")
except B.BgrpoError as e:
    assert e.status == B.ERR_CAPACITY, e.status
B.tree_sync_status(s.tree)                               # the word is cleared by the read
print("debug-bounds build: status clean after", len(cases), "workloads; tripped check reported")
'''


def _debug_env():
    env = dict(os.environ)
    env["BGRPO_DEBUG_BOUNDS"] = "1"
    return env


def test_status_stays_clean_under_the_index_checking_build():
    import __graft_entry__
    __graft_entry__.build()
    out = subprocess.run([sys.executable, "-c", SCRIPT], cwd=ROOT, env=_debug_env(), capture_output=True, text=True, timeout=900)
    assert out.returncode == 0, out.stdout[-2000:] + out.stderr[-4000:]
    assert "tripped check reported" in out.stdout


def test_normal_build_says_it_has_no_index_checks():
    import __graft_entry__
    __graft_entry__.build()
    from paper_2509_06040_b200 import binding as B
    if B.DEBUG_BOUNDS:
        pytest.skip("this process loaded the debug build")
    with pytest.raises(B.BgrpoError) as e:
        B.debug_bounds(None)
    assert e.value.status == B.ERR_UNSUPPORTED


def test_parity_tests_pass_against_the_index_checking_build():
    out = subprocess.run([sys.executable, "-m", "pytest", "tests/test_gpu_parity.py", "tests/test_gpu_mlp.py", "-m", "gpu", "-x", "-q",
                          "-k", "toy or rollout_parity or fused_rollout_matches or logprob or leaf_rewards or mlp_stage_matches or prune_masks"],
                         cwd=ROOT, env=_debug_env(), capture_output=True, text=True, timeout=1800)
    assert out.returncode == 0, out.stdout[-4000:] + out.stderr[-2000:]
