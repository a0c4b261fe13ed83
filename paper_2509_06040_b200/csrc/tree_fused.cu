// Whole-tree rollout in one launch, for velocities that act on each latent element by itself (the closed-form linear
// Gaussian-target velocity).  With such a velocity an element's trajectory through the tree never looks at any other
// element, so a thread can carry its elements from the root through every depth in registers, depth first, and
// write each node's latent exactly once: the parent read of the level-by-level step kernel disappears (4 bytes per
// element and node-step instead of 8) and the T launches become one.  The saving the Branch Rollout Algorithm draws
// from shared prefixes is taken literally: a prefix is computed once and never re-read.
//
// Every node gets exactly the value the level-by-level path gives it: the same Philox counters (element block, global
// node id, step, tag), the same float32 expressions (mean = ca z + cb mu, child = g xi + mean, Eq. 2 noise mixing).
// Log-prob sums use their own partial layout (one float per node row and warp of the CTAs that cover the row) and are
// completed by finalize_tree_kernel in a fixed order, in double.
#include "internal.h"
#include "philox.cuh"

namespace bgrpo {
namespace {

struct Ctx {
    uint32_t e[kFusedVec];        // float4 index of each of this thread's pieces
    bool live[kFusedVec];         // inside the row
    float4 mu[kFusedVec];
    float4* tree_base;            // latents of this tree, as float4
    int64_t tree_row0;            // first row of this tree in the per-node buffers
    uint32_t gid0;                // global node id of the tree's local node 0
    int chunk, warp, lane;
    bool writes_table;            // one thread per tree appends the node-table rows
};

__device__ __forceinline__ float4 fma4(float a, const float4& x, const float4& y) {
    return make_float4(fmaf(a, x.x, y.x), fmaf(a, x.y, y.y), fmaf(a, x.z, y.z), fmaf(a, x.w, y.w));
}

// One child: z' = mean + g xi, its latent row, its squared residual partial, its node-table row.
__device__ __forceinline__ void emit_child(const FusedLaunch& p, const Ctx& cx, int step, int parent_local, int child_local,
                                           int split_step, int branch_id, float g, const float4 (&m)[kFusedVec],
                                           const float4 (&xi0)[kFusedVec], bool shared, float4 (&c)[kFusedVec]) {
    const uint32_t gid = cx.gid0 + static_cast<uint32_t>(child_local);
    if (!BGRPO_IN_BOUNDS(p.status, child_local > 0 && child_local < p.nodes_cap && parent_local >= 0 && parent_local < child_local &&
                                       (cx.chunk + 1) * (kFusedThreads / 32) <= p.per_row_cap)) return;
    float acc = 0.0f;
    float4* row = cx.tree_base + static_cast<size_t>(child_local) * static_cast<size_t>(p.D >> 2);
#pragma unroll
    for (int k = 0; k < kFusedVec; ++k) {
        if (cx.live[k]) {
            float4 xi = make_float4(0.f, 0.f, 0.f, 0.f);
            if (g != 0.0f) {
                xi = noise4(cx.e[k], gid, static_cast<uint32_t>(step), BGRPO_TAG_INNOV, p.keys);
                if (shared) {
                    xi.x = fmaf(p.mix_innov, xi.x, p.mix_shared * xi0[k].x);
                    xi.y = fmaf(p.mix_innov, xi.y, p.mix_shared * xi0[k].y);
                    xi.z = fmaf(p.mix_innov, xi.z, p.mix_shared * xi0[k].z);
                    xi.w = fmaf(p.mix_innov, xi.w, p.mix_shared * xi0[k].w);
                }
            }
            c[k] = fma4(g, xi, m[k]);
            __stcs(row + cx.e[k], c[k]);
            // z' - mean is g xi up to the rounding of z': sum xi^2, times g^2 once per warp
            acc = fmaf(xi.x, xi.x, acc);
            acc = fmaf(xi.y, xi.y, acc);
            acc = fmaf(xi.z, xi.z, acc);
            acc = fmaf(xi.w, xi.w, acc);
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_down_sync(0xffffffffu, acc, o);
    acc *= g * g;
    const int64_t r = cx.tree_row0 + child_local;
    if (cx.lane == 0) p.partialsf[r * p.per_row + cx.chunk * (kFusedThreads / 32) + cx.warp] = acc;
    if (cx.writes_table) {
        const int64_t rows = static_cast<int64_t>(p.n_trees) * p.nodes_cap;
        p.table[r] = parent_local;
        p.table[rows + r] = step + 1;
        p.table[2 * rows + r] = split_step;
        p.table[3 * rows + r] = branch_id;
    }
}

// Walks the subtree below local node j of depth i, whose latent pieces are in z.  S counts the splits on the path so
// far: each split level keeps its parent's mean in registers while the children's subtrees are walked one by one.
// MAXS bounds the number of split levels the instantiation walks, SHARED says whether split steps mix in a per-parent
// xi_0 (finite s): the common case (few splits, independent children) then carries neither the deeper levels' code nor
// registers for xi_0.
template <int S, int MAXS, bool SHARED>
__device__ __forceinline__ void walk(const FusedLaunch& p, const Ctx& cx, int i, int j, int split_step, int branch_id,
                                     float4 (&z)[kFusedVec]) {
    const float4 zero[kFusedVec] = {};
    for (; i < p.T; ++i) {
        const float ca = p.ca[i], cb = p.cb[i], g = p.g[i];
        float4 m[kFusedVec];
#pragma unroll
        for (int k = 0; k < kFusedVec; ++k)
            m[k] = make_float4(fmaf(ca, z[k].x, cb * cx.mu[k].x), fmaf(ca, z[k].y, cb * cx.mu[k].y),
                               fmaf(ca, z[k].z, cb * cx.mu[k].z), fmaf(ca, z[k].w, cb * cx.mu[k].w));
        const int parent_local = p.off[i] + j;
        if (!((p.split_bits >> i) & 1ull)) {
            emit_child(p, cx, i, parent_local, p.off[i + 1] + j, split_step, branch_id, g, m, zero, false, z);
            continue;
        }
        if constexpr (S < MAXS) {
            const bool shared = SHARED && g != 0.0f;
            float4 xi0[kFusedVec] = {};
            if (shared) {
#pragma unroll
                for (int k = 0; k < kFusedVec; ++k)
                    if (cx.live[k])
                        xi0[k] = noise4(cx.e[k], cx.gid0 + static_cast<uint32_t>(parent_local), static_cast<uint32_t>(i), BGRPO_TAG_SHARED, p.keys);
            }
            for (int b = 0; b < p.K; ++b) {
                float4 c[kFusedVec];
                const int child = j * p.K + b;
                emit_child(p, cx, i, parent_local, p.off[i + 1] + child, i, b, g, m, xi0, shared, c);
                walk<S + 1, MAXS, SHARED>(p, cx, i + 1, child, i, b, c);
            }
        }
        return;
    }
}

template <int MAXS, bool SHARED>
__global__ void __launch_bounds__(kFusedThreads)
rollout_fused_kernel(const __grid_constant__ FusedLaunch p) {
    pdl_release();
    pdl_wait();
    Ctx cx;
    cx.chunk = blockIdx.x % p.nchunks;
    const int tree = blockIdx.x / p.nchunks;
    cx.warp = threadIdx.x >> 5;
    cx.lane = threadIdx.x & 31;
    cx.tree_row0 = static_cast<int64_t>(tree) * p.nodes_cap;
    cx.gid0 = p.node_id_base + static_cast<uint32_t>(cx.tree_row0);
    cx.tree_base = reinterpret_cast<float4*>(p.latents + cx.tree_row0 * p.D);
    cx.writes_table = (cx.chunk == 0 && threadIdx.x == 0);
    const uint32_t D4 = static_cast<uint32_t>(p.D >> 2);
    const float4* __restrict__ mu = reinterpret_cast<const float4*>(p.mu + static_cast<int64_t>(tree) * p.D);
    float4 z[kFusedVec];
#pragma unroll
    for (int k = 0; k < kFusedVec; ++k) {
        cx.e[k] = static_cast<uint32_t>(cx.chunk) * kFusedChunkVec + k * kFusedThreads + threadIdx.x;
        cx.live[k] = cx.e[k] < D4;
        cx.mu[k] = make_float4(0.f, 0.f, 0.f, 0.f);
        z[k] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (cx.live[k]) {
            cx.mu[k] = __ldg(mu + cx.e[k]);
            z[k] = __ldcs(cx.tree_base + cx.e[k]);          // root latent (row 0 of the tree)
        }
    }
    walk<0, MAXS, SHARED>(p, cx, 0, 0, -1, 0, z);
}

// Completes the log-probs of every non-root node of every tree from the fused kernel's partial sums: one warp per node
// row, lanes stride over the row's per_row floats in index order, then a fixed shuffle tree; double
// throughout.
__global__ void __launch_bounds__(256)
finalize_tree_kernel(const __grid_constant__ FusedLaunch p, int32_t nodes) {
    pdl_release();
    pdl_wait();
    const int lane = threadIdx.x & 31;
    const int64_t w = static_cast<int64_t>(blockIdx.x) * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int64_t total = static_cast<int64_t>(p.n_trees) * (nodes - 1);
    if (w >= total) return;
    const int tree = static_cast<int>(w / (nodes - 1));
    const int local = 1 + static_cast<int>(w - static_cast<int64_t>(tree) * (nodes - 1));
    int step = 0;                                       // the node's depth is step + 1
    while (step + 1 < p.T && local >= p.off[step + 2]) ++step;
    const int64_t row = static_cast<int64_t>(tree) * p.nodes_cap + local;
    const int per_row = p.per_row;
    if (!BGRPO_IN_BOUNDS(p.status, local < p.nodes_cap && per_row <= p.per_row_cap)) return;
    const float* q = p.partialsf + row * per_row;
    double s = 0.0;
    for (int c = lane; c < per_row; c += 32) s += static_cast<double>(__ldcg(q + c));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_down_sync(0xffffffffu, s, o);
    if (lane == 0) {
        const float g = p.g[step];
        p.logp[row] = (g == 0.0f) ? 0.0f
                                   : static_cast<float>(-(s / static_cast<double>(p.D)) * static_cast<double>(p.inv_2g2[step]) +
                                                        static_cast<double>(p.logp_const[step]));
    }
}

}  // namespace

cudaError_t launch_rollout_fused(const FusedLaunch& p, int32_t nodes, cudaStream_t s) {
    const int64_t items = static_cast<int64_t>(p.n_trees) * p.nchunks;
    if (items <= 0 || items > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
    const unsigned int grid = static_cast<unsigned int>(items);
    const int n_splits = __builtin_popcountll(p.split_bits);
    if (n_splits > kFusedMaxSplits) return cudaErrorInvalidValue;
    cudaError_t e;
    if (p.shared_noise) {
        if (n_splits <= 3) e = launch_overlapped(rollout_fused_kernel<3, true>, grid, kFusedThreads, 0, s, p);
        else e = launch_overlapped(rollout_fused_kernel<kFusedMaxSplits, true>, grid, kFusedThreads, 0, s, p);
    } else {
        if (n_splits <= 3) e = launch_overlapped(rollout_fused_kernel<3, false>, grid, kFusedThreads, 0, s, p);
        else e = launch_overlapped(rollout_fused_kernel<kFusedMaxSplits, false>, grid, kFusedThreads, 0, s, p);
    }
    if (e != cudaSuccess || nodes < 2) return e;
    const int64_t warps = static_cast<int64_t>(p.n_trees) * (nodes - 1);
    return launch_overlapped(finalize_tree_kernel, static_cast<unsigned int>((warps + 7) / 8), 256, 0, s, p, nodes);
}

}  // namespace bgrpo
