"""The C-ABI library loads, exports every symbol the header declares, and its host-only entry
points and argument checks behave; no kernel is launched here."""
import ctypes
import math
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def B():
    import __graft_entry__
    __graft_entry__.build()
    from paper_2509_06040_b200 import binding
    return binding


def test_every_declared_symbol_is_exported(B):
    header = open(os.path.join(ROOT, "include", "bgrpo.h")).read()
    names = set(re.findall(r"\b(bgrpo_[a-z_0-9]+)\s*\(", header))
    names -= {"bgrpo_status"}
    assert len(names) >= 20
    for n in names:
        assert hasattr(B.lib, n), n
    assert names == set(B._SIGNATURES), names ^ set(B._SIGNATURES)


def test_struct_layouts_match_header(B):
    assert ctypes.sizeof(B.TreeDesc) == 56 and B.TreeDesc.t_grid.offset == 48 and B.TreeDesc.seed.offset == 40
    assert ctypes.sizeof(B.Buffers) == 64 and ctypes.sizeof(B.Sizes) == 40


def test_tree_count_matches_paper_nfe(B):
    c = B.tree_count(20, 2, [0, 3, 6, 9])
    assert c == dict(nodes=219, node_steps=218, model_evals=203, leaves=16)
    assert abs(c["nodes"] / c["leaves"] - 13.68) < 0.01          # Table 1, BranchGRPO row
    assert B.tree_count(20, 3, [0, 3, 6, 9])["leaves"] == 81
    assert B.tree_count(16, 2, [])["nodes"] == 17
    with pytest.raises(B.BgrpoError):
        B.tree_count(20, 2, [3, 3])
    with pytest.raises(B.BgrpoError):
        B.tree_count(20, 5, [1])


def test_workspace_and_argument_checks(B):
    from workloads import CONFIGS
    w = CONFIGS["image"]
    desc, grid = B.make_desc(1, w.tokens, w.channels, w.T, w.K, w.nodes, 0.3, w.t_grid(), 7)
    sz = B.tree_workspace(desc)
    assert sz.latents_bytes == 155 * 129600 * 4 and sz.node_table_bytes == 4 * 155 * 4 and sz.mask_bytes == 155
    assert sz.scratch_bytes >= 256 + 155 * 4 + 155 * 32 * 3 * 8
    bad, _ = B.make_desc(1, 3, 1, 4, 2, 20, 0.3, np.linspace(1, 0, 5), 7)       # D % 4 != 0
    with pytest.raises(B.BgrpoError) as e:
        B.tree_workspace(bad)
    assert e.value.status == B.ERR_INVALID_ARG
    for kw in (dict(T=0), dict(T=65), dict(K=5), dict(nodes_cap=3), dict(sigma=-1.0)):
        args = dict(n_trees=1, tokens=16, channels=4, T=4, K=2, nodes_cap=13, sigma=0.3)
        args.update(kw)
        d, _ = B.make_desc(args["n_trees"], args["tokens"], args["channels"], args["T"], args["K"], args["nodes_cap"],
                           args["sigma"], np.linspace(1, 0, max(args["T"], 1) + 1), 7)
        with pytest.raises(B.BgrpoError):
            B.tree_workspace(d)


def test_init_rejects_null_buffers_without_touching_a_gpu(B):
    desc, grid = B.make_desc(1, 16, 4, 4, 2, 13, 0.3, np.linspace(1, 0, 5), 7)
    h = ctypes.c_void_p()
    st = B.lib.bgrpo_tree_init(ctypes.byref(desc), ctypes.byref(B.Buffers()), None, ctypes.byref(h))
    assert st == B.ERR_INVALID_ARG and not h.value
    assert b"NULL" in B.lib.bgrpo_last_error()
    assert B.lib.bgrpo_tree_step(None, 0, None, None) == B.ERR_INVALID_ARG
    assert B.lib.bgrpo_status_string(B.ERR_CAPACITY) == b"capacity exceeded"


def test_depth_window_matches_the_stated_schedule(B):
    assert B.depth_window(0, 9) == [9, 10, 11, 12]
    assert B.depth_window(30, 9) == [10, 11, 12, 13]
    assert B.depth_window(3000, 9, stop=16) == [12, 13, 14, 15]
    from oracle import credit
    for it in (0, 29, 31, 95, 400):
        assert B.depth_window(it, 9, 4, 30, 16) == credit.depth_window(it, 9, 4, 30, 16)
    with pytest.raises(B.BgrpoError):
        B.depth_window(0, 9, size=0)


def test_mlp_packed_bytes(B):
    assert B.velocity_mlp_packed_bytes(3072) >= 2 * 64 * 3072 * 2
    assert B.velocity_mlp_packed_bytes(100) == 0


def test_binding_refuses_to_import_without_the_library(tmp_path):
    """There is no CPU or PyTorch fallback: a copy of the package without libbgrpo.so fails at import, loudly."""
    import shutil
    import subprocess
    import sys
    pkg = tmp_path / "paper_2509_06040_b200"
    pkg.mkdir()
    src = os.path.join(ROOT, "paper_2509_06040_b200")
    for name in ("__init__.py", "binding.py", "session.py"):
        shutil.copy(os.path.join(src, name), pkg / name)
    out = subprocess.run([sys.executable, "-c", "import paper_2509_06040_b200.binding"], cwd=tmp_path, capture_output=True, text=True,
                         env={k: v for k, v in os.environ.items() if k != "PYTHONPATH"})
    assert out.returncode != 0
    assert "libbgrpo.so is missing" in out.stderr and "no CPU or PyTorch fallback" in out.stderr
