"""bgrpo_reward_mse_static: the leaf-reward reduction for callers that cannot allocate device memory where they
call the library (all memory already given to their own pool, or a cudaMalloc there would stall the whole device).
It keeps its reduction scratch in an array built into the library, so this test checks, through the C ABI, that it
returns what the ordinary entry point (bgrpo_leaf_reward_mse, caller-allocated scratch) returns and what the CPU oracle
computes from the same rows - on several calls in a row with different shapes, because the built-in array is shared by
all calls and keeps the previous call's contents - and that sizes beyond the built-in array are refused.  The file name makes pytest collect it last."""
import numpy as np
import pytest
import torch

from workloads import Workload, make_inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    import __graft_entry__
    __graft_entry__.build()
    from paper_2509_06040_b200 import binding
    assert torch.cuda.is_available()
    return binding


def _leaf_rewards_both_ways(B, tokens, K, splits, seed):
    from paper_2509_06040_b200.session import TreeSession
    w = Workload(name="static", n_trees=1, tokens=tokens, channels=4, T=3, K=K, splits=splits, sigma=0.3,
                 velocity="linear", reward="neg_mse_target", seed=seed)
    s = TreeSession(w)
    s.upload_inputs(make_inputs(w))
    s.rollout()
    s.rewards()                                             # existing entry point: bgrpo_leaf_reward_mse
    widths, offsets = B.tree_levels(s.tree)
    leaves, off_leaf = widths[-1], offsets[-1]
    rows = s.latents[0, off_leaf:off_leaf + leaves]          # the leaf rows are contiguous in the pool
    out = torch.full((leaves,), float("nan"), device="cuda")
    B.reward_mse_static(rows, s.target[0], leaves, w.D, out)
    torch.cuda.synchronize()
    from oracle import rewards
    rows_h, target_h = rows.cpu().numpy(), s.target[0].cpu().numpy()
    oracle = np.array([rewards.neg_mse(rows_h[i], target_h) for i in range(leaves)])
    return s.leaf_r[0].cpu().numpy(), out.cpu().numpy(), oracle


def test_static_scratch_matches_caller_scratch_on_two_calls_in_a_row(B):
    # first call: 9 rows of 3 chunks with a ragged tail; second call: 4 rows of 1 chunk - fewer rows and chunks
    # than the call before, so stale partials and counters from the first call sit right beside the live ones
    for tokens, K, splits, seed in ((2125, 3, (0, 2), 5), (300, 2, (0, 1), 6), (2125, 3, (0, 2), 7)):
        ref, got, oracle = _leaf_rewards_both_ways(B, tokens, K, splits, seed)
        assert np.all(np.isfinite(got))
        assert np.abs(got - ref).max() <= 1e-6 * max(1.0, np.abs(ref).max())
        assert np.abs(got - oracle).max() <= 1e-6 * max(1.0, np.abs(oracle).max())


def test_sizes_beyond_the_built_in_array_are_refused(B):
    x = torch.zeros(16, device="cuda")
    out = torch.full((4,), 3.0, device="cuda")
    for n_rows, D in ((B.STATIC_MAX_ROWS + 1, 4), (1024, 4096 * 64), (2, 4096 * 40000)):
        with pytest.raises(B.BgrpoError) as e:
            B.reward_mse_static(x, x, n_rows, D, out)       # refused before any pointer is touched
        assert e.value.status == B.ERR_CAPACITY
    with pytest.raises(B.BgrpoError) as e:
        B.reward_mse_static(x, x, 1, 6, out)
    assert e.value.status == B.ERR_INVALID_ARG
    torch.cuda.synchronize()
    assert torch.all(out == 3.0)
