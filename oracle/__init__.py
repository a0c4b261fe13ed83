"""CPU oracle for the BranchGRPO tree rollout and tree reductions.

TEST INFRASTRUCTURE ONLY.  This package is a plain, slow, fp64 restatement of
what the paper defines (branch sampling Eq. 2 and the appendix "Branch Noise
Construction", reward fusion Eq. 3, depth-wise normalisation Eq. 4, the
pruning rules of the "Pruning Strategies" section, the NFE convention of
Table 1).  It exists to check the CUDA library and to be timed as a CPU
baseline; nothing in the product path may import it, and it imports nothing
from the CUDA package.

Modules
-------
philox   counter-based noise: Philox4x32-10, uniform map, Box-Muller normals
tree     level-order rollout tree: node table, widths, NFE accounting
sde      Euler-Maruyama flow-SDE step, branch noise, transition log-prob, rollout
mlp      bf16-emulating per-token MLP velocity
credit   reward fusion, depth-wise advantages, width/depth pruning masks
rewards  leaf-reward stand-ins (-MSE, cosine)

Pins: every function is pinned by tests/test_oracle_*.py against values the
paper prints, closed forms, library routines or brute force.  Parity unpinned:
the *choice* of drift discretisation (rectified-flow score form, see sde.py)
and of the per-element-mean normalisation of the log-prob are readings the
paper's text cannot confirm; they are pinned only through the marginal-
preservation property the paper claims and through library log-densities.
"""
