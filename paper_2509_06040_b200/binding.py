"""ctypes binding of libbgrpo.so: argument marshalling only.

Every function here has the name of the C entry point it calls (without the
``bgrpo_`` prefix) and does nothing but turn torch tensors into device
pointers, python numbers into C scalars, and status codes into exceptions.
All arithmetic of the method runs in the CUDA kernels behind the C ABI
declared in include/bgrpo.h; there is no CPU fallback, and importing this
module fails if the shared library has not been built.
"""
from __future__ import annotations

import ctypes as C
import math
import os
from dataclasses import dataclass
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
# BGRPO_DEBUG_BOUNDS=1 selects the build whose kernels check every index they derive (python -m ...build --debug-bounds)
DEBUG_BOUNDS = os.environ.get("BGRPO_DEBUG_BOUNDS", "0") == "1"
LIB_PATH = os.path.join(_HERE, "libbgrpo_debug.so" if DEBUG_BOUNDS else "libbgrpo.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python -m paper_2509_06040_b200.build` "
        "(the library has no CPU or PyTorch fallback)")
lib = C.CDLL(LIB_PATH)

OK, ERR_INVALID_ARG, ERR_STATE, ERR_CAPACITY, ERR_NONFINITE, ERR_CUDA, ERR_UNSUPPORTED = range(7)
WIDTH_NONE, WIDTH_PER_SPLIT_TOPK, WIDTH_LAST_SPLIT_TOPK, WIDTH_EXTREME_B = range(4)
TAG_ROOT, TAG_SHARED, TAG_INNOV = range(3)
MAX_T, MAX_K = 64, 4


class BgrpoError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        detail = lib.bgrpo_last_error().decode()
        super().__init__(f"{where}: {lib.bgrpo_status_string(status).decode()} ({detail})")


class TreeDesc(C.Structure):
    _fields_ = [("n_trees", C.c_int32), ("tokens", C.c_int32), ("channels", C.c_int32), ("T", C.c_int32),
                ("K", C.c_int32), ("nodes_cap", C.c_int32), ("tree_id_base", C.c_int64), ("sigma", C.c_float),
                ("branch_corr_s", C.c_float), ("seed", C.c_uint64), ("t_grid", C.POINTER(C.c_float))]


class Buffers(C.Structure):
    _fields_ = [("latents", C.c_void_p), ("node_table", C.c_void_p), ("logp", C.c_void_p), ("rbar", C.c_void_p),
                ("adv", C.c_void_p), ("mask", C.c_void_p), ("scratch", C.c_void_p), ("scratch_bytes", C.c_size_t)]


class Sizes(C.Structure):
    _fields_ = [("latents_bytes", C.c_size_t), ("node_table_bytes", C.c_size_t), ("per_node_float_bytes", C.c_size_t),
                ("mask_bytes", C.c_size_t), ("scratch_bytes", C.c_size_t)]


_i32p, _i64p, _f32p = C.POINTER(C.c_int32), C.POINTER(C.c_int64), C.POINTER(C.c_float)
_SIGNATURES = {
    "bgrpo_tree_workspace": (C.c_int, [C.POINTER(TreeDesc), C.POINTER(Sizes)]),
    "bgrpo_tree_count": (C.c_int, [C.c_int32, C.c_int32, _i32p, C.c_int32, _i64p, _i64p, _i64p, _i64p]),
    "bgrpo_tree_init": (C.c_int, [C.POINTER(TreeDesc), C.POINTER(Buffers), C.c_void_p, C.POINTER(C.c_void_p)]),
    "bgrpo_tree_reset": (C.c_int, [C.c_void_p, C.c_uint64, C.c_void_p]),
    "bgrpo_velocity_linear_bind": (C.c_int, [C.c_void_p, C.c_void_p, C.c_float]),
    "bgrpo_tree_step": (C.c_int, [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p]),
    "bgrpo_tree_rollout": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p]),
    "bgrpo_tree_rollout_fused": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p]),
    "bgrpo_tree_logprob": (C.c_int, [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p]),
    "bgrpo_velocity_mlp_packed_bytes": (C.c_size_t, [C.c_int32]),
    "bgrpo_velocity_mlp_pack": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p]),
    "bgrpo_velocity_mlp": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p]),
    "bgrpo_leaf_reward_mse": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "bgrpo_leaf_reward_cos": (C.c_int, [C.c_void_p, C.c_void_p, C.c_float, C.c_void_p, C.c_void_p]),
    "bgrpo_tree_fuse_advantage": (C.c_int, [C.c_void_p, C.c_void_p, C.c_float, C.c_float, C.c_float, C.c_float, C.c_void_p]),
    "bgrpo_tree_fusion_ess": (C.c_int, [C.c_void_p, C.c_float, C.c_float, C.c_void_p, C.c_void_p]),
    "bgrpo_tree_prune": (C.c_int, [C.c_void_p, C.c_int32, C.c_int32, _i32p, C.c_int32, C.c_int32, C.c_void_p]),
    "bgrpo_tree_grpo_objective": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_float, C.c_float, C.c_void_p, C.c_void_p, C.c_void_p]),
    "bgrpo_tree_set_sde_steps": (C.c_int, [C.c_void_p, C.c_void_p]),
    "bgrpo_mix_sde_steps": (C.c_int, [C.c_int32, _i32p, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_void_p]),
    "bgrpo_depth_window": (C.c_int, [C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_int32, _i32p, _i32p]),
    "bgrpo_tree_stats": (C.c_int, [C.c_void_p, _i32p, _i64p, _i64p, _i64p, _i64p]),
    "bgrpo_tree_levels": (C.c_int, [C.c_void_p, C.c_int32, _i32p, _i32p]),
    "bgrpo_tree_sync_status": (C.c_int, [C.c_void_p, C.c_void_p]),
    "bgrpo_philox_words_fill": (C.c_int, [C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint32, C.c_void_p, C.c_int64, C.c_void_p]),
    "bgrpo_philox_normal_fill": (C.c_int, [C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint32, C.c_void_p, C.c_int64, C.c_void_p]),
    "bgrpo_reward_mse_static": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int32, C.c_int64, C.c_void_p, C.c_void_p]),
    "bgrpo_tree_export_bytes": (C.c_size_t, []),
    "bgrpo_tree_export": (C.c_int, [C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]),
    "bgrpo_tree_import": (C.c_int, [C.c_void_p, C.c_size_t, C.POINTER(Buffers), C.c_void_p, C.POINTER(C.c_void_p)]),
    "bgrpo_debug_bounds": (C.c_int, [C.c_void_p, C.c_int32, C.c_void_p]),
    "bgrpo_tree_destroy": (None, [C.c_void_p]),
    "bgrpo_status_string": (C.c_char_p, [C.c_int]),
    "bgrpo_last_error": (C.c_char_p, []),
}
for _name, (_res, _args) in _SIGNATURES.items():
    _fn = getattr(lib, _name)       # AttributeError here = the library does not export a declared symbol
    _fn.restype, _fn.argtypes = _res, _args


def _check(status: int, where: str):
    if status != OK:
        raise BgrpoError(status, where)


def _ptr(t) -> Optional[int]:
    """Device (or host) address of a torch tensor / numpy array; None stays NULL."""
    if t is None:
        return None
    if isinstance(t, np.ndarray):
        return t.ctypes.data
    assert t.is_contiguous(), "tensors crossing the C ABI must be contiguous"
    return t.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        import torch
        if not torch.cuda.is_available():
            return None
        return torch.cuda.current_stream().cuda_stream or None
    return getattr(stream, "cuda_stream", stream) or None


@dataclass
class Tree:
    """Opaque handle plus the objects that must stay alive while it is used."""
    handle: int
    desc: TreeDesc
    keep: tuple

    def __del__(self):
        if getattr(self, "handle", None) and lib is not None:     # `lib` is gone at interpreter shutdown
            lib.bgrpo_tree_destroy(self.handle)
            self.handle = None


def make_desc(n_trees, tokens, channels, T, K, nodes_cap, sigma, t_grid, seed, branch_corr_s=math.inf, tree_id_base=0):
    grid = np.ascontiguousarray(t_grid, dtype=np.float32)
    d = TreeDesc(n_trees, tokens, channels, T, K, nodes_cap, tree_id_base, sigma, branch_corr_s, seed,
                 grid.ctypes.data_as(_f32p))
    return d, grid


def tree_workspace(desc: TreeDesc) -> Sizes:
    s = Sizes()
    _check(lib.bgrpo_tree_workspace(C.byref(desc), C.byref(s)), "bgrpo_tree_workspace")
    return s


def tree_count(T: int, K: int, split_steps: Sequence[int]):
    arr = (C.c_int32 * max(1, len(split_steps)))(*split_steps)
    out = [C.c_int64() for _ in range(4)]
    _check(lib.bgrpo_tree_count(T, K, arr, len(split_steps), *[C.byref(o) for o in out]), "bgrpo_tree_count")
    return dict(zip(("nodes", "node_steps", "model_evals", "leaves"), (o.value for o in out)))


def tree_init(desc: TreeDesc, latents, node_table, logp, rbar, adv, mask, scratch, stream=None, keep=()) -> Tree:
    b = Buffers(_ptr(latents), _ptr(node_table), _ptr(logp), _ptr(rbar), _ptr(adv), _ptr(mask), _ptr(scratch),
                scratch.numel() * scratch.element_size())
    h = C.c_void_p()
    _check(lib.bgrpo_tree_init(C.byref(desc), C.byref(b), _stream(stream), C.byref(h)), "bgrpo_tree_init")
    return Tree(h.value, desc, (latents, node_table, logp, rbar, adv, mask, scratch) + tuple(keep))


def tree_reset(tree: Tree, seed: int, stream=None):
    _check(lib.bgrpo_tree_reset(tree.handle, seed, _stream(stream)), "bgrpo_tree_reset")


def velocity_linear_bind(tree: Tree, mu, s0: float):
    _check(lib.bgrpo_velocity_linear_bind(tree.handle, _ptr(mu), s0), "bgrpo_velocity_linear_bind")
    tree.keep = tree.keep + (mu,)


def tree_step(tree: Tree, split_flag: int, v=None, stream=None):
    _check(lib.bgrpo_tree_step(tree.handle, int(split_flag), _ptr(v), _stream(stream)), "bgrpo_tree_step")


def tree_rollout(tree: Tree, split_flags, packed=None, hidden: int = 0, v=None, stream=None):
    """split_flags: a numpy uint8 array of T flags (kept by the caller) or any sequence."""
    arr = split_flags if isinstance(split_flags, np.ndarray) and split_flags.dtype == np.uint8 else \
        np.ascontiguousarray([1 if f else 0 for f in split_flags], dtype=np.uint8)
    _check(lib.bgrpo_tree_rollout(tree.handle, arr.ctypes.data, _ptr(packed), hidden, _ptr(v), _stream(stream)), "bgrpo_tree_rollout")


def tree_rollout_fused(tree: Tree, split_flags: Sequence[int], stream=None):
    arr = np.ascontiguousarray([1 if f else 0 for f in split_flags], dtype=np.uint8)
    _check(lib.bgrpo_tree_rollout_fused(tree.handle, arr.ctypes.data, _stream(stream)), "bgrpo_tree_rollout_fused")


def tree_logprob(tree: Tree, step: int, v, logp_out, stream=None):
    _check(lib.bgrpo_tree_logprob(tree.handle, step, _ptr(v), _ptr(logp_out), _stream(stream)), "bgrpo_tree_logprob")


def velocity_mlp_packed_bytes(hidden: int) -> int:
    return lib.bgrpo_velocity_mlp_packed_bytes(hidden)


def velocity_mlp_pack(W1_bf16, W2_bf16, hidden: int, packed, stream=None):
    _check(lib.bgrpo_velocity_mlp_pack(_ptr(W1_bf16), _ptr(W2_bf16), hidden, _ptr(packed), _stream(stream)),
           "bgrpo_velocity_mlp_pack")


def velocity_mlp(tree: Tree, packed, hidden: int, v_out, stream=None):
    _check(lib.bgrpo_velocity_mlp(tree.handle, _ptr(packed), hidden, _ptr(v_out), _stream(stream)), "bgrpo_velocity_mlp")


def leaf_reward_mse(tree: Tree, target, r_out, stream=None):
    _check(lib.bgrpo_leaf_reward_mse(tree.handle, _ptr(target), _ptr(r_out), _stream(stream)), "bgrpo_leaf_reward_mse")


def leaf_reward_cos(tree: Tree, target, scale: float, r_inout, stream=None):
    _check(lib.bgrpo_leaf_reward_cos(tree.handle, _ptr(target), scale, _ptr(r_inout), _stream(stream)),
           "bgrpo_leaf_reward_cos")


def tree_fuse_advantage(tree: Tree, leaf_rewards, beta=0.0, logp_scale=1.0, eps=1e-6, adv_clip_max=0.0, stream=None):
    _check(lib.bgrpo_tree_fuse_advantage(tree.handle, _ptr(leaf_rewards), beta, logp_scale, eps, adv_clip_max,
                                         _stream(stream)), "bgrpo_tree_fuse_advantage")


def tree_fusion_ess(tree: Tree, beta: float, logp_scale: float, ess_out, stream=None):
    _check(lib.bgrpo_tree_fusion_ess(tree.handle, beta, logp_scale, _ptr(ess_out), _stream(stream)), "bgrpo_tree_fusion_ess")


def tree_prune(tree: Tree, width_mode: int, k_or_b: int, pruned_steps: Sequence[int] = (), ignore_last_step=False,
               stream=None):
    n = len(pruned_steps)
    arr = (C.c_int32 * max(1, n))(*[int(x) for x in pruned_steps])
    _check(lib.bgrpo_tree_prune(tree.handle, width_mode, k_or_b, arr, n, int(bool(ignore_last_step)), _stream(stream)),
           "bgrpo_tree_prune")


def tree_grpo_objective(tree: Tree, logp_new, logp_old=None, logp_scale=1.0, clip_eps=1e-4, terms_out=None, J_out=None,
                        stream=None):
    _check(lib.bgrpo_tree_grpo_objective(tree.handle, _ptr(logp_new), _ptr(logp_old), logp_scale, clip_eps, _ptr(terms_out),
                                         _ptr(J_out), _stream(stream)), "bgrpo_tree_grpo_objective")


def tree_set_sde_steps(tree: Tree, sde_flags: Optional[Sequence[int]]):
    arr = None if sde_flags is None else np.ascontiguousarray(sde_flags, dtype=np.uint8)
    _check(lib.bgrpo_tree_set_sde_steps(tree.handle, None if arr is None else arr.ctypes.data), "bgrpo_tree_set_sde_steps")


def mix_sde_steps(T: int, split_steps: Sequence[int], iteration: int, window: int = 4, every: int = 30, start: int = 0):
    arr = (C.c_int32 * max(1, len(split_steps)))(*[int(x) for x in split_steps])
    out = np.zeros(T, dtype=np.uint8)
    _check(lib.bgrpo_mix_sde_steps(T, arr, len(split_steps), iteration, window, every, start, out.ctypes.data), "bgrpo_mix_sde_steps")
    return [i for i in range(T) if out[i]]


def depth_window(iteration: int, start: int, size: int = 4, every: int = 30, stop: int = -1):
    out = (C.c_int32 * max(1, size))()
    n = C.c_int32()
    _check(lib.bgrpo_depth_window(iteration, start, size, every, stop, out, C.byref(n)), "bgrpo_depth_window")
    return [out[i] for i in range(n.value)]


def tree_stats(tree: Tree):
    d = C.c_int32()
    out = [C.c_int64() for _ in range(4)]
    _check(lib.bgrpo_tree_stats(tree.handle, C.byref(d), *[C.byref(o) for o in out]), "bgrpo_tree_stats")
    return dict(depth=d.value, nodes=out[0].value, node_steps=out[1].value, model_evals=out[2].value,
                frontier_width=out[3].value)


def tree_levels(tree: Tree):
    n = MAX_T + 1
    w, o = (C.c_int32 * n)(), (C.c_int32 * n)()
    _check(lib.bgrpo_tree_levels(tree.handle, n, w, o), "bgrpo_tree_levels")
    depth = tree_stats(tree)["depth"]
    return [w[i] for i in range(depth + 1)], [o[i] for i in range(depth + 1)]


def tree_sync_status(tree: Tree, stream=None):
    _check(lib.bgrpo_tree_sync_status(tree.handle, _stream(stream)), "bgrpo_tree_sync_status")


def tree_export(tree: Tree, stream=None) -> bytes:
    buf = C.create_string_buffer(lib.bgrpo_tree_export_bytes())
    _check(lib.bgrpo_tree_export(tree.handle, buf, len(buf), _stream(stream)), "bgrpo_tree_export")
    return buf.raw


def tree_import(blob: bytes, latents, node_table, logp, rbar, adv, mask, scratch, stream=None, keep=()) -> Tree:
    b = Buffers(_ptr(latents), _ptr(node_table), _ptr(logp), _ptr(rbar), _ptr(adv), _ptr(mask), _ptr(scratch),
                scratch.numel() * scratch.element_size())
    h = C.c_void_p()
    _check(lib.bgrpo_tree_import(blob, len(blob), C.byref(b), _stream(stream), C.byref(h)), "bgrpo_tree_import")
    return Tree(h.value, None, (latents, node_table, logp, rbar, adv, mask, scratch) + tuple(keep))


def debug_bounds(tree: Optional[Tree], trip: bool = False, stream=None):
    """OK only in the build with device-side index checks; trip=True also makes one check fail on purpose."""
    _check(lib.bgrpo_debug_bounds(tree.handle if tree is not None else None, int(bool(trip)), _stream(stream)), "bgrpo_debug_bounds")


def philox_words_fill(seed, node_id, step, tag, out, n_blocks, stream=None):
    _check(lib.bgrpo_philox_words_fill(seed, node_id, step, tag, _ptr(out), n_blocks, _stream(stream)),
           "bgrpo_philox_words_fill")


def philox_normal_fill(seed, node_id, step, tag, out, n, stream=None):
    _check(lib.bgrpo_philox_normal_fill(seed, node_id, step, tag, _ptr(out), n, _stream(stream)),
           "bgrpo_philox_normal_fill")


STATIC_SCRATCH_BYTES, STATIC_MAX_ROWS = 512 * 1024, 1024


def reward_mse_static(rows, target, n_rows: int, D: int, r_out, stream=None):
    """-MSE of n_rows latent rows against one target, using the library's built-in scratch array instead of a
    caller-allocated one (for callers that cannot allocate device memory when they call).  Raises BgrpoError
    (ERR_CAPACITY) when n_rows or n_rows * ceil(D/4096) is beyond what the built-in array holds."""
    _check(lib.bgrpo_reward_mse_static(_ptr(rows), _ptr(target), n_rows, D, _ptr(r_out), _stream(stream)),
           "bgrpo_reward_mse_static")
