// Leaf-reward stand-ins (Algorithm 1, "Evaluate rewards"; the paper's reward models are out of scope): streaming
// reductions over the leaf rows.  Sums over a row are float32 over runs of sixteen elements, double from there on, one
// double per (row, chunk, component), and the chunks are added in a fixed order by a small finish kernel.
#include "internal.h"

namespace bgrpo {
namespace {

constexpr int kWarps = kStreamThreads / 32;
constexpr int kPartialStride = 3;                           // doubles per (row, chunk) slot
constexpr int kBatch = 8;                                   // float4 of each operand a thread has in flight at once
constexpr int kBatches = kRewardVec / kBatch;

__device__ __forceinline__ double warp_sum(double x) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_down_sync(0xffffffffu, x, o);
    return x;
}

// Sum of one component of a row's chunk partials, in chunk order within each lane and a fixed shuffle tree across
// lanes.  Called by whole warps only.
__device__ __forceinline__ double row_total(const double* partials, int64_t row, int comp, int nchunks) {
    const int lane = threadIdx.x & 31;
    double s = 0.0;
    for (int c = lane; c < nchunks; c += 32) s += __ldcg(&partials[(row * nchunks + c) * kPartialStride + comp]);
    s = warp_sum(s);
    return __shfl_sync(0xffffffffu, s, 0);
}

// ---------------------------------------------------------------------------------------------------------------
// Leaf rewards: mode 0  r = -mean (z - target)^2 ; mode 1  r += scale * cos(z, target).
// One CTA per (leaf row, chunk of kRewardChunkVec float4 = 64 KiB of the row).  A thread takes sixteen float4 of the row
// and of the target in two batches of eight; the sixteen 128-bit loads of a batch are issued before the first value is
// used.  Sums are float32 over a run of sixteen elements (four float4), double from there on; the warp and CTA
// reductions, in double, happen once per 64 KiB, so they cost a few per cent of the instructions instead of most of them.
// 128-bit loads as volatile instructions: the compiler keeps the loads of a batch in program order, ahead of the
// arithmetic that uses them, instead of sinking each load to its first use.  The leaf row is read once (evict first);
// the target row is shared by all leaves of a tree (read-only path).
__device__ __forceinline__ float4 load_streaming(const float4* p) {
    float4 v;
    asm volatile("ld.global.cs.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ float4 load_shared_row(const float4* p) {
    float4 v;
    asm volatile("ld.global.nc.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p));
    return v;
}

// FULL: the chunk lies inside the row, no element needs a bounds test (so the loads of a batch are plain back-to-back
// instructions the compiler keeps together).
template <int MODE, bool FULL>
__device__ __forceinline__ void accumulate_chunk(const float4* __restrict__ z, const float4* __restrict__ tg, uint32_t e0, uint32_t D4,
                                                 double (&dsum)[(MODE == 0) ? 1 : 3]) {
    constexpr int NV = (MODE == 0) ? 1 : 3;
#pragma unroll
    for (int h = 0; h < kBatches; ++h) {
        float4 a[kBatch], t[kBatch];
#pragma unroll
        for (int k = 0; k < kBatch; ++k) {
            const uint32_t e = e0 + static_cast<uint32_t>(h * kBatch + k) * kStreamThreads;
            if (FULL || e < D4) {
                a[k] = load_streaming(z + e);
                t[k] = load_shared_row(tg + e);
            } else {
                a[k] = make_float4(0.f, 0.f, 0.f, 0.f);      // past the row: contributes nothing to any of the sums
                t[k] = make_float4(0.f, 0.f, 0.f, 0.f);
            }
        }
        if (FULL) {      // nothing below may move above the last load of the batch
#pragma unroll
            for (int k = 0; k < kBatch; ++k) {
                asm volatile("" : "+f"(a[k].x), "+f"(a[k].y), "+f"(a[k].z), "+f"(a[k].w));
                asm volatile("" : "+f"(t[k].x), "+f"(t[k].y), "+f"(t[k].z), "+f"(t[k].w));
            }
        }
#pragma unroll
        for (int run = 0; run < kBatch / 4; ++run) {         // sixteen elements in float32, then into the double
            float acc[NV];
#pragma unroll
            for (int v = 0; v < NV; ++v) acc[v] = 0.0f;
#pragma unroll
            for (int k = run * 4; k < run * 4 + 4; ++k) {
                const float av[4] = {a[k].x, a[k].y, a[k].z, a[k].w};
                const float tv[4] = {t[k].x, t[k].y, t[k].z, t[k].w};
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    if (MODE == 0) {
                        const float d = av[q] - tv[q];
                        acc[0] = fmaf(d, d, acc[0]);
                    } else {
                        acc[0] = fmaf(av[q], tv[q], acc[0]);
                        acc[1] = fmaf(av[q], av[q], acc[1]);
                        acc[2] = fmaf(tv[q], tv[q], acc[2]);
                    }
                }
            }
#pragma unroll
            for (int v = 0; v < NV; ++v) dsum[v] += static_cast<double>(acc[v]);
        }
    }
}

// Three or four CTAs per SM: with that many registers to spend the compiler keeps a batch's loads ahead of its
// arithmetic (left to aim at full occupancy it sinks every load to its first use, and the kernel waits on one 128-bit load
// at a time; measured 70.7 us at full occupancy against 54.3 us here on 512 rows of 129 600 elements).
template <int MODE>
__global__ void __launch_bounds__(kStreamThreads, MODE == 0 ? 3 : 4)
reward_kernel(const __grid_constant__ RewardLaunch p) {
    pdl_release();
    pdl_wait();
    const int chunk = blockIdx.x % p.nchunks;
    const int row = blockIdx.x / p.nchunks;             // tree * leaves + l
    const int tree = row / p.leaves;
    const int l = row - tree * p.leaves;
    const uint32_t D4 = static_cast<uint32_t>(p.D >> 2);
    const int64_t node_row = static_cast<int64_t>(tree) * p.nodes_cap + p.off_leaf + l;
    const float4* __restrict__ z = reinterpret_cast<const float4*>(p.latents + node_row * p.D);
    const float4* __restrict__ tg = reinterpret_cast<const float4*>(p.target + static_cast<int64_t>(tree) * p.D);
    constexpr int NV = (MODE == 0) ? 1 : 3;
    const uint32_t c0 = static_cast<uint32_t>(chunk) * kRewardChunkVec;
    if (!BGRPO_IN_BOUNDS(p.status, tree < p.n_trees && p.off_leaf + l < p.nodes_cap && c0 < D4 && p.nchunks <= p.nchunks_cap)) return;
    double dsum[NV];
#pragma unroll
    for (int v = 0; v < NV; ++v) dsum[v] = 0.0;
    if (c0 + kRewardChunkVec <= D4) accumulate_chunk<MODE, true>(z, tg, c0 + threadIdx.x, D4, dsum);
    else accumulate_chunk<MODE, false>(z, tg, c0 + threadIdx.x, D4, dsum);
    // One double per (row, chunk, component).  Nothing waits for these stores; reward_finish_kernel, next on the
    // stream, adds the chunks up in order.
    __shared__ double red[NV][kWarps];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int v = 0; v < NV; ++v) {
        const double s = warp_sum(dsum[v]);
        if (lane == 0) red[v][warp] = s;
    }
    __syncthreads();
    if (threadIdx.x < NV) {
        double s = 0.0;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) s += red[threadIdx.x][w];
        p.partials[(node_row * p.nchunks + chunk) * kPartialStride + threadIdx.x] = s;
    }
}

// One warp per leaf row: the row's chunk partials in chunk order within each lane, a fixed shuffle tree across lanes.
template <int MODE>
__global__ void __launch_bounds__(kStreamThreads)
reward_finish_kernel(const __grid_constant__ RewardLaunch p) {
    pdl_release();
    pdl_wait();
    const int row = blockIdx.x * (kStreamThreads / 32) + (threadIdx.x >> 5);      // tree * leaves + l
    if (row >= p.n_trees * p.leaves) return;
    const int tree = row / p.leaves;
    const int64_t node_row = static_cast<int64_t>(tree) * p.nodes_cap + p.off_leaf + (row - tree * p.leaves);
    if (!BGRPO_IN_BOUNDS(p.status, p.off_leaf + p.leaves <= p.nodes_cap && p.nchunks <= p.nchunks_cap)) return;
    if (MODE == 0) {
        const double ss = row_total(p.partials, node_row, 0, p.nchunks);
        if ((threadIdx.x & 31) == 0) p.r[row] = static_cast<float>(-ss / static_cast<double>(p.D));
    } else {
        const double dot = row_total(p.partials, node_row, 0, p.nchunks);
        const double zz = row_total(p.partials, node_row, 1, p.nchunks);
        const double tt = row_total(p.partials, node_row, 2, p.nchunks);
        if ((threadIdx.x & 31) == 0)
            p.r[row] = static_cast<float>(static_cast<double>(p.r[row]) + static_cast<double>(p.scale) * dot / (sqrt(zz) * sqrt(tt)));
    }
}

}  // namespace

cudaError_t launch_reward(const RewardLaunch& p, cudaStream_t s) {
    const int64_t items = static_cast<int64_t>(p.n_trees) * p.leaves * p.nchunks;
    if (items <= 0 || items > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
    const unsigned int rows = static_cast<unsigned int>(p.n_trees) * static_cast<unsigned int>(p.leaves);
    const unsigned int fgrid = (rows + kStreamThreads / 32 - 1) / (kStreamThreads / 32);
    cudaError_t e;
    if (p.mode == 0) {
        e = launch_overlapped(reward_kernel<0>, static_cast<unsigned int>(items), kStreamThreads, 0, s, p);
        if (e == cudaSuccess) e = launch_overlapped(reward_finish_kernel<0>, fgrid, kStreamThreads, 0, s, p);
    } else {
        e = launch_overlapped(reward_kernel<1>, static_cast<unsigned int>(items), kStreamThreads, 0, s, p);
        if (e == cudaSuccess) e = launch_overlapped(reward_finish_kernel<1>, fgrid, kStreamThreads, 0, s, p);
    }
    return e;
}

}  // namespace bgrpo
