// Leaf-reward stand-ins (Algorithm 1, "Evaluate rewards"; the paper's reward models are out of scope): streaming
// reductions over the leaf rows.  Sums over a row are float32 inside a thread, double from the warp level on, one double
// per (row, chunk, component), and the chunks are added in a fixed order by a small finish kernel.
#include "internal.h"

namespace bgrpo {
namespace {

constexpr int kVecPerThread = kChunkVec / kStreamThreads;   // 4
constexpr int kWarps = kStreamThreads / 32;
constexpr int kPartialStride = 3;                           // doubles per (row, chunk) slot
constexpr int kPairs = 1;                                   // chunks per CTA of the reward kernel (1 and 2 measured the same)

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
template <int MODE>
__global__ void __launch_bounds__(kStreamThreads)
reward_kernel(const __grid_constant__ RewardLaunch p) {
    pdl_release();
    pdl_wait();
    // A CTA takes kPairs consecutive chunks of a row and issues all their loads before it touches a value.
    const int npairs = (p.nchunks + kPairs - 1) / kPairs;
    const int pair = blockIdx.x % npairs;
    const int row = blockIdx.x / npairs;                // tree * leaves + l
    const int tree = row / p.leaves;
    const int l = row - tree * p.leaves;
    const int64_t D4 = p.D >> 2;
    const int64_t node_row = static_cast<int64_t>(tree) * p.nodes_cap + p.off_leaf + l;
    const float4* __restrict__ z = reinterpret_cast<const float4*>(p.latents + node_row * p.D);
    const float4* __restrict__ tg = reinterpret_cast<const float4*>(p.target + static_cast<int64_t>(tree) * p.D);
    constexpr int NV = (MODE == 0) ? 1 : 3;
    float acc[kPairs][NV];
    float4 a[kPairs][kVecPerThread], t[kPairs][kVecPerThread];
#pragma unroll
    for (int h = 0; h < kPairs; ++h) {
#pragma unroll
        for (int v = 0; v < NV; ++v) acc[h][v] = 0.0f;
        const int64_t e0 = static_cast<int64_t>(pair * kPairs + h) * kChunkVec + threadIdx.x;
#pragma unroll
        for (int k = 0; k < kVecPerThread; ++k) {
            const int64_t e = e0 + k * kStreamThreads;
            if (e < D4) { a[h][k] = __ldcs(z + e); t[h][k] = __ldg(tg + e); }
        }
    }
#pragma unroll
    for (int h = 0; h < kPairs; ++h) {
        const int64_t e0 = static_cast<int64_t>(pair * kPairs + h) * kChunkVec + threadIdx.x;
#pragma unroll
        for (int k = 0; k < kVecPerThread; ++k) {
            const int64_t e = e0 + k * kStreamThreads;
            if (e < D4) {
                const float av[4] = {a[h][k].x, a[h][k].y, a[h][k].z, a[h][k].w};
                const float tv[4] = {t[h][k].x, t[h][k].y, t[h][k].z, t[h][k].w};
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    if (MODE == 0) {
                        const float d = av[q] - tv[q];
                        acc[h][0] = fmaf(d, d, acc[h][0]);
                    } else {
                        acc[h][0] = fmaf(av[q], tv[q], acc[h][0]);
                        acc[h][1] = fmaf(av[q], av[q], acc[h][1]);
                        acc[h][2] = fmaf(tv[q], tv[q], acc[h][2]);
                    }
                }
            }
        }
    }
    // One double per (row, chunk, component): thread sums are float over 16 elements, double from the warp level on.
    // Nothing waits for these stores; reward_finish_kernel, next on the stream, adds the chunks up in order.
    __shared__ double red[kPairs * NV][kWarps];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int h = 0; h < kPairs; ++h)
#pragma unroll
        for (int v = 0; v < NV; ++v) {
            const double s = warp_sum(static_cast<double>(acc[h][v]));
            if (lane == 0) red[h * NV + v][warp] = s;
        }
    __syncthreads();
    if (threadIdx.x < kPairs * NV) {
        const int h = threadIdx.x / NV, v = threadIdx.x - h * NV;
        const int chunk = pair * kPairs + h;
        if (chunk < p.nchunks) {
            double s = 0.0;
#pragma unroll
            for (int w = 0; w < kWarps; ++w) s += red[threadIdx.x][w];
            p.partials[(node_row * p.nchunks + chunk) * kPartialStride + v] = s;
        }
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
    const int64_t items = static_cast<int64_t>(p.n_trees) * p.leaves * ((p.nchunks + kPairs - 1) / kPairs);
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
