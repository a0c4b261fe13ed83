"""B200-native tree rollout and tree reductions of BranchGRPO (C ABI in include/bgrpo.h).

``binding`` marshals torch tensors into the C entry points; ``session`` sequences those
calls for a named workload.  The shared library must be built first
(``python -m paper_2509_06040_b200.build``); nothing here computes on the CPU.
"""
