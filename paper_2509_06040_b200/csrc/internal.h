// Host-side state of a batch of rollout trees and the launch interfaces of the kernels.
#pragma once
#include <cstddef>
#include <cstdint>
#include <cuda_runtime.h>
#include <utility>

#include "../../include/bgrpo.h"

namespace bgrpo {

constexpr int kStreamThreads = 256;    // threads per CTA of the root / reward kernels
constexpr int kChunkVec = 1024;        // float4 per (row, chunk) work item of the root kernel
constexpr int kRewardVec = 16;         // float4 of a row per thread of the leaf-reward kernel
constexpr int kRewardChunkVec = kStreamThreads * kRewardVec;   // float4 per (row, chunk) work item of the leaf-reward kernel
// Step kernel: 64-thread CTAs, 8 float4 per thread.  Measured on B200 against 128/256-thread CTAs, 2/4/6 float4 per
// thread, persistent grids and a shared-memory ring fed by bulk asynchronous copies: the kernel is bound by
// instruction issue (Philox + Box-Muller), and eight independent noise chains per thread with many small CTAs
// per SM gave the best rate on both the 8 B/element and the 12 B/element workloads.
constexpr int kStepThreads = 64;
constexpr int kStepVec = 8;
constexpr int kStepChunkVec = kStepThreads * kStepVec;   // 512 float4 = 8 KiB per operand tile
constexpr int kStepWarps = kStepThreads / 32;            // log-prob partials per (row, chunk)
constexpr int kStepCtasPerSm = 8;
// Whole-tree rollout kernel: 128-thread CTAs, 2 float4 per thread (measured on B200 against 64/256 threads and 1/2/4
// float4: within 6 % of one another), one log-prob partial per node row and warp; at most kFusedMaxSplits split steps
// (one register-resident parent mean per split level on the depth-first walk).
constexpr int kFusedThreads = 128;
constexpr int kFusedVec = 2;
constexpr int kFusedChunkVec = kFusedThreads * kFusedVec;   // float4 of a row per CTA
constexpr int kFusedMaxSplits = 6;
// log-prob partials of the whole-tree kernel per node row: one float per warp of every CTA that covers the row
inline int64_t fused_partials_per_row(int64_t D) { return ((D / 4 + kFusedChunkVec - 1) / kFusedChunkVec) * (kFusedThreads / 32); }
// floats of log-prob partials reserved per node row: the larger of the two rollout kernels' layouts
inline int64_t partials_per_row(int64_t D) {
    const int64_t D4 = D / 4;
    const int64_t step = ((D4 + kStepChunkVec - 1) / kStepChunkVec) * kStepWarps;
    const int64_t fused = fused_partials_per_row(D);
    return step > fused ? step : fused;
}
constexpr int kScratchHeader = 256;    // bytes reserved at the start of scratch for the status word

constexpr uint32_t kPhiloxM0 = 0xD2511F53u;   // Philox4x32 multipliers and Weyl key increments (Salmon et al., SC'11)
constexpr uint32_t kPhiloxM1 = 0xCD9E8D57u;
constexpr uint32_t kPhiloxW0 = 0x9E3779B9u;
constexpr uint32_t kPhiloxW1 = 0xBB67AE85u;

// The ten round keys of a 64-bit seed: key r = (k0 + r*W0, k1 + r*W1).  They are the same for every thread of
// a launch, so the host computes them once and the kernels read them as launch constants.
struct PhiloxKeys {
    uint32_t k[10][2];
};

inline PhiloxKeys make_philox_keys(uint64_t seed) {
    PhiloxKeys out;
    uint32_t k0 = static_cast<uint32_t>(seed), k1 = static_cast<uint32_t>(seed >> 32);
    for (int r = 0; r < 10; ++r) {
        out.k[r][0] = k0;
        out.k[r][1] = k1;
        k0 += kPhiloxW0;
        k1 += kPhiloxW1;
    }
    return out;
}

// Per-step scalars of the Euler-Maruyama mean and the Gaussian transition, computed in double on the host.
//   mean = a*z + b*v                       (v given)
//        = lin_a*z + lin_b*mu              (closed-form velocity v = k z - (1 + k(1-t)) mu folded in)
struct StepCoef {
    float a, b;          // a = 1 - c, b = -(h + c (1-t)), c = sigma^2 h / (2 t)
    float lin_a, lin_b;  // valid once a linear velocity is bound
    float g;             // sigma sqrt(h)
    float inv_2g2;       // 1 / (2 g^2), 0 when g == 0
    float logp_const;    // -ln g - 0.5 ln(2 pi), 0 when g == 0
};

// Log-probs of a level whose per-(row, chunk, warp) partial sums are in scratch but not yet added up.  The sum is
// taken by the next kernel the library enqueues on the stream (the next step's prologue, or a small flush kernel).
struct FinalizeDesc {
    float* logp_out;       // nullptr: nothing pending
    int32_t W, off;        // rows off .. off+W-1 of every tree
    float g, inv_2g2, logp_const;
};

struct LevelInfo {                       // layout of the tree grown so far
    int32_t width[BGRPO_MAX_T + 1];
    int32_t offset[BGRPO_MAX_T + 2];
    int32_t fanout[BGRPO_MAX_T];         // children per node produced by step i (K or 1)
};

}  // namespace bgrpo

struct bgrpo_tree {
    bgrpo_tree_desc desc;
    bgrpo_buffers buf;
    float t_grid[BGRPO_MAX_T + 1];
    bgrpo::StepCoef coef[BGRPO_MAX_T];
    bgrpo::LevelInfo lv;
    uint64_t ode_bits;                   // bit i set: step i is an ODE step of the hybrid schedule (sigma = 0)
    int32_t depth;                       // steps taken so far
    int64_t D;                           // elements per node
    int32_t nchunks;                     // root-kernel work items per node row (also sizes the reward partials)
    int32_t nchunks_reward;              // leaf-reward work items per node row
    int32_t nchunks_step;                // step-kernel work items per node row
    bool independent;                    // s = inf: xi_b = eta_b
    float mix_shared, mix_innov;         // xi_b = mix_shared*xi_0 + mix_innov*eta_b
    const float* mu;                     // bound linear velocity (device), or nullptr
    float s0;
    // scratch carving (device pointers inside buf.scratch)
    int32_t* status;
    unsigned int* counters;              // one ticket counter per (tree, node row)
    double* partials;                    // [n_trees*nodes_cap][nchunks][3]   (reward reductions)
    double* node_scratch;                // [n_trees][2][nodes_cap]: per-node state of the tree reductions when a tree
                                         // is too large for one CTA's shared memory
    float* partialsf;                    // [n_trees*nodes_cap][partials_per_row] (log-prob sums of the rollout kernels)
    unsigned int* mlp_tickets;           // 64-channel trees only: scratch of the MLP stage's split over the hidden dimension
    float* mlp_partials;
    bgrpo::FinalizeDesc pending;         // level whose log-probs still have to be summed
};

// Debug build (-DBGRPO_DEBUG_BOUNDS): every kernel tests the row, chunk and element indices it derives against the
// extents it was launched with, before the access.  A failed test sets bit 2 of the tree's status word and the access
// is skipped; nothing traps.  bgrpo_tree_sync_status reports the word.  In the normal build the tests compile to nothing.
#ifdef BGRPO_DEBUG_BOUNDS
#define BGRPO_IN_BOUNDS(status, cond) ((cond) ? true : (atomicOr((status), 2), false))
#else
#define BGRPO_IN_BOUNDS(status, cond) true
#endif
constexpr int kStatusNonFinite = 1, kStatusOutOfBounds = 2, kStatusWaitTimeout = 4;

namespace bgrpo {

// Programmatic dependent launch: a kernel launched with launch_overlapped() may be scheduled while the kernel before it
// on the stream is still draining, so the gap between two dependent launches shrinks to the set-up the new kernel can do
// on its own.  Such a kernel calls pdl_wait() before it touches anything an earlier kernel wrote or still reads, and
// pdl_release() as early as it likes to let its own successor in.
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_release() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
template <typename... Params, typename... Args>
cudaError_t launch_overlapped(void (*kernel)(Params...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}
#endif

// ---- streaming kernels (tree_step.cu) -------------------------------------------------------------------------
struct StepLaunch {
    float* latents;
    const float* v;            // [n_trees][W_in][D] or nullptr
    const float* mu;           // [n_trees][D] or nullptr
    float* logp;
    int32_t* table;            // SoA, stride = n_trees*nodes_cap
    int64_t D;                 // elements per row
    int32_t n_trees, nodes_cap, nchunks;   // nchunks: step-kernel chunks per row
    int32_t W_in, off_in, off_out, fan, step, is_split;
    uint32_t node_id_base;     // tree_id_base * nodes_cap
    PhiloxKeys keys;
    float ca, cb;              // mean = ca*z + cb*x, x = v or mu
    float g, inv_2g2, logp_const;
    float mix_shared, mix_innov;
    int32_t shared_noise;      // 1: finite s at a split step
    int32_t write_children;    // 1: tree_step; 0: tree_logprob (children are read, nothing but logp is written)
    float* logp_out;           // destination of the log-probs (== logp for tree_step)
    int32_t* status;           // the tree's status word
    int32_t per_row;           // floats reserved per node row in partialsf
    float* partialsf;          // [rows][nchunks][kStepWarps] warp sums of (z' - mean)^2
    FinalizeDesc prev;         // level to finalize in this launch's prologue (logp_out == nullptr: none)
};
cudaError_t launch_root(const bgrpo_tree* t, cudaStream_t s);
cudaError_t launch_step(const StepLaunch& p, cudaStream_t s);
cudaError_t launch_finalize(const bgrpo_tree* t, const FinalizeDesc& f, cudaStream_t s);

struct RewardLaunch {
    const float* latents; const float* target; float* r; double* partials; unsigned int* counters; int32_t* status;
    int64_t D; int32_t n_trees, nodes_cap, nchunks, nchunks_cap, leaves, off_leaf; float scale; int32_t mode;  // 0 mse, 1 cos; nchunks_cap: partial slots reserved per row
};
cudaError_t launch_reward(const RewardLaunch& p, cudaStream_t s);

cudaError_t launch_philox_words(uint64_t seed, uint32_t node, uint32_t step, uint32_t tag, uint32_t* out, int64_t nblk, cudaStream_t s);
cudaError_t launch_philox_normals(uint64_t seed, uint32_t node, uint32_t step, uint32_t tag, float* out, int64_t n, cudaStream_t s);

// ---- whole-tree rollout (tree_fused.cu) -------------------------------------------------------------------------
struct FusedLaunch {
    float* latents;
    const float* mu;           // [n_trees][D]
    float* logp;
    int32_t* table;
    float* partialsf;          // [rows][per_row]: one float per warp of the CTAs that cover a row
    int32_t* status;           // the tree's status word
    int32_t per_row_cap;       // floats reserved per node row in partialsf
    int64_t D;
    int32_t n_trees, nodes_cap, nchunks, per_row, T, K, shared_noise;   // nchunks: CTAs per tree
    uint32_t node_id_base;
    uint64_t split_bits;       // bit i: step i forks every node into K children
    PhiloxKeys keys;
    float mix_shared, mix_innov;
    int32_t off[BGRPO_MAX_T + 2];                      // first local index of every depth
    float ca[BGRPO_MAX_T], cb[BGRPO_MAX_T], g[BGRPO_MAX_T], inv_2g2[BGRPO_MAX_T], logp_const[BGRPO_MAX_T];
};
cudaError_t launch_rollout_fused(const FusedLaunch& p, int32_t nodes, cudaStream_t s);

// ---- tree reductions (tree_reduce.cu) -------------------------------------------------------------------------
constexpr size_t kTreeSmemLimit = 200 * 1024;   // per-node doubles beyond this live in node_scratch instead of shared memory
struct FuseLaunch {
    const float* leaf_r; const float* logp; float* rbar; float* adv; int32_t* status;
    double* node_scratch;      // [n_trees][2][nodes_cap], used when three doubles per node exceed kTreeSmemLimit (trees of more than 8 533 nodes)
    LevelInfo lv; int32_t n_trees, nodes_cap, T, nodes; double beta_scaled; float eps, clip;
};
cudaError_t launch_fuse_advantage(const FuseLaunch& p, cudaStream_t s);

struct EssLaunch {
    const float* logp; float* ess; double* node_scratch; int32_t* status;
    LevelInfo lv; int32_t n_trees, nodes_cap, T, nodes; double beta_scaled;
};
cudaError_t launch_fusion_ess(const EssLaunch& p, cudaStream_t s);

struct PruneLaunch {
    const float* rbar; const int32_t* table; uint8_t* mask; int32_t* status;
    LevelInfo lv; int32_t n_trees, nodes_cap, T, nodes, mode, k, last_split, ignore_last, values_in_smem; uint64_t pruned_bits;
};
cudaError_t launch_prune(const PruneLaunch& p, cudaStream_t s);

struct ObjectiveLaunch {
    const float* logp_new; const float* logp_old; const float* adv; const uint8_t* mask; float* terms; float* J; int32_t* status;
    int32_t n_trees, nodes_cap, nodes; double logp_scale; float clip_eps;
};
cudaError_t launch_objective(const ObjectiveLaunch& p, cudaStream_t s);

// ---- MLP velocity (mlp_velocity.cu) -----------------------------------------------------------------------------
// Frontiers of fewer tiles than SMs are also cut along the hidden dimension; the partial output tiles (128 tokens x 64
// channels, float) of at most this many CTAs and one ticket counter per tile live in the tree's scratch.
constexpr int kMlpSplitMaxCtas = 192;
constexpr size_t kMlpPartialBytes = static_cast<size_t>(kMlpSplitMaxCtas) * 128 * 64 * sizeof(float);
constexpr size_t kMlpTicketBytes = 1024;      // kMlpSplitMaxCtas counters, rounded up
size_t mlp_packed_bytes(int hidden);
cudaError_t launch_mlp_pack(const uint16_t* W1, const uint16_t* W2, int hidden, void* packed, cudaStream_t s);
cudaError_t launch_debug_trip(int32_t* status, cudaStream_t s);     // debug build: fails one index test on purpose (no access involved)
cudaError_t launch_mlp(const float* latents, int64_t pool_elems, int64_t tree_stride, int64_t row_offset, int n_trees, int64_t tokens_per_tree,
                       const void* packed, int hidden, float* v_out, float* split_partials, unsigned int* split_tickets,
                       int32_t* status, cudaStream_t s);

}  // namespace bgrpo
