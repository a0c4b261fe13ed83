// Streaming kernels of the rollout: root initialisation, the fused gather / fork / Euler-Maruyama update /
// log-prob step (Eq. 2 and the appendix's Euler-Maruyama form) and the log-prob recompute under a given velocity.  All of them are HBM-bound: every latent element is read or written once,
// with 128-bit accesses, and the noise is generated in registers.
//
// Sums over a row are float32 inside a thread (inside a warp for the step's log-prob), double from there on, and
// always added in a fixed order, so results do not depend on scheduling.
#include "internal.h"
#include "philox.cuh"

namespace bgrpo {
namespace {

constexpr int kVecPerThread = kChunkVec / kStreamThreads;   // 4
constexpr int kWarps = kStreamThreads / 32;

__device__ __forceinline__ double warp_sum(double x) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_down_sync(0xffffffffu, x, o);
    return x;
}

// ---------------------------------------------------------------------------------------------------------------
// Root: z_0 ~ N(0, I) from the ROOT stream, node-table row of the root, and a clean scratch (counters, status).
__global__ void __launch_bounds__(kStreamThreads)
root_kernel(float* latents, int32_t* table, float* logp, unsigned int* counters, int32_t* status, int64_t D,
            int32_t n_trees, int32_t nodes_cap, int32_t nchunks, uint32_t node_id_base, const __grid_constant__ PhiloxKeys keys) {
    pdl_release();
    pdl_wait();           // the buffers may still be read by the kernels of the previous pass
    const int chunk = blockIdx.x % nchunks;
    const int tree = blockIdx.x / nchunks;
    const int64_t D4 = D >> 2;
    if (!BGRPO_IN_BOUNDS(status, tree < n_trees && static_cast<int64_t>(chunk) * kChunkVec < D4)) return;
    float4* z = reinterpret_cast<float4*>(latents + static_cast<int64_t>(tree) * nodes_cap * D);
    const uint32_t gid = node_id_base + static_cast<uint32_t>(tree) * nodes_cap;
#pragma unroll
    for (int k = 0; k < kVecPerThread; ++k) {
        const int64_t e = static_cast<int64_t>(chunk) * kChunkVec + k * kStreamThreads + threadIdx.x;
        if (e < D4) z[e] = noise4(static_cast<uint32_t>(e), gid, 0u, BGRPO_TAG_ROOT, keys);
    }
    const int64_t rows = static_cast<int64_t>(n_trees) * nodes_cap;
    if (chunk == 0) {
        for (int n = threadIdx.x; n < nodes_cap; n += kStreamThreads) counters[static_cast<int64_t>(tree) * nodes_cap + n] = 0u;
        if (threadIdx.x == 0) {
            const int64_t r = static_cast<int64_t>(tree) * nodes_cap;
            table[r] = -1;
            table[rows + r] = 0;
            table[2 * rows + r] = -1;
            table[3 * rows + r] = 0;
            logp[r] = 0.0f;
            if (tree == 0) *status = 0;
        }
    }
}

// ---------------------------------------------------------------------------------------------------------------
// Fused step.  One CTA of kStepThreads threads per work item (tree, parent, chunk of kStepChunkVec float4).
//
// A thread issues the 128-bit loads of its kStepVec float4 of the parent tile and of the operand tile (velocity or
// target mean) first, then generates the noise of all its elements - Philox and Box-Muller depend on indices only,
// so kStepVec independent chains per child are in flight while the loads travel - and only then touches the loaded
// values: mean once per parent element, then for each of the K children z' = mean + g xi (128-bit store) and the
// squared residual.  The parent is read once however many children it has.
//
// Log-prob: a warp adds its squared residuals per child in float with a fixed shuffle tree and stores one float per
// (child row, chunk, warp).  Nothing waits for those stores: the sums over chunks and warps are taken, in double and
// in a fixed order, by the prologue of the NEXT launch on the stream (FinalizeDesc), or by the small flush kernel
// when the tree is complete, so the kernel has no fence, no atomic and no CTA-wide barrier.
//
// FAN children per parent; SHARED: xi_b mixes a per-parent xi_0 (finite s at a split step); WRITE: true =
// tree_step (draw noise, write children), false = tree_logprob (read children, score them); FULL: the tile holds
// kStepChunkVec float4, so no element needs a bounds test; NOISY = false: a deterministic step (sigma = 0) of the
// hybrid schedule, no noise is generated at all.

// Adds up the pending level's partial sums: one warp per row, lanes stride over the row's nchunks * kStepWarps floats
// in index order, then a fixed shuffle tree; double throughout.
__device__ __forceinline__ void finalize_rows(const FinalizeDesc& f, const float* partialsf, int32_t n_trees, int32_t nodes_cap,
                                              int32_t nchunks, int64_t D, int warp_global, int warps_total, int32_t* status, int32_t per_row_cap) {
    const int lane = threadIdx.x & 31;
    const int n_rows = n_trees * f.W;
    const int per_row = nchunks * kStepWarps;
    for (int idx = warp_global; idx < n_rows; idx += warps_total) {
        const int tree = idx / f.W;
        const int64_t row = static_cast<int64_t>(tree) * nodes_cap + f.off + (idx - tree * f.W);
        if (!BGRPO_IN_BOUNDS(status, f.off + f.W <= nodes_cap && per_row <= per_row_cap)) continue;
        const float* q = partialsf + row * per_row;
        double s = 0.0;
        for (int c = lane; c < per_row; c += 32) s += static_cast<double>(__ldcg(q + c));
        s = warp_sum(s);
        if (lane == 0)
            f.logp_out[row] = (f.g == 0.0f) ? 0.0f
                                            : static_cast<float>(-(s / static_cast<double>(D)) * static_cast<double>(f.inv_2g2) +
                                                                 static_cast<double>(f.logp_const));
    }
}

template <bool FULL>
__device__ __forceinline__ void load_tile(const float4* __restrict__ zp, const float4* __restrict__ xop, bool streamed,
                                          uint32_t vecs, float4 (&z)[kStepVec], float4 (&x)[kStepVec]) {
#pragma unroll
    for (int k = 0; k < kStepVec; ++k) {
        const uint32_t t = threadIdx.x + k * kStepThreads;
        if (FULL || t < vecs) {
            z[k] = __ldcs(zp + t);                                   // read once: evict first
            x[k] = streamed ? __ldcs(xop + t) : __ldg(xop + t);      // the target mean is shared by the whole level
        }
    }
}

template <int FAN, bool SHARED, bool WRITE, bool FULL, bool NOISY>
__device__ __forceinline__ void compute_tile(const StepLaunch& p, const float4 (&z)[kStepVec], const float4 (&x)[kStepVec],
                                             uint32_t vecs, uint32_t e_base, uint32_t D4, float4* zc, uint32_t gid_parent,
                                             uint32_t gid_child0, float (&acc)[FAN]) {
#pragma unroll
    for (int k = 0; k < kStepVec; ++k) {
        const uint32_t t = threadIdx.x + k * kStepThreads;
        if (FULL || t < vecs) {
            const uint32_t e = e_base + t;
            float4 xi[FAN];
            if (WRITE && !NOISY) {       // deterministic step (sigma = 0): no noise is drawn, the child is the mean
#pragma unroll
                for (int b = 0; b < FAN; ++b) xi[b] = make_float4(0.f, 0.f, 0.f, 0.f);
            } else if (WRITE) {
                float4 xi0 = make_float4(0.f, 0.f, 0.f, 0.f);
                if (SHARED) xi0 = noise4(e, gid_parent, p.step, BGRPO_TAG_SHARED, p.keys);
#pragma unroll
                for (int b = 0; b < FAN; ++b) {
                    xi[b] = noise4(e, gid_child0 + b, p.step, BGRPO_TAG_INNOV, p.keys);
                    if (SHARED) {
                        xi[b].x = fmaf(p.mix_innov, xi[b].x, p.mix_shared * xi0.x);
                        xi[b].y = fmaf(p.mix_innov, xi[b].y, p.mix_shared * xi0.y);
                        xi[b].z = fmaf(p.mix_innov, xi[b].z, p.mix_shared * xi0.z);
                        xi[b].w = fmaf(p.mix_innov, xi[b].w, p.mix_shared * xi0.w);
                    }
                }
            }
            float4 m;
            m.x = fmaf(p.ca, z[k].x, p.cb * x[k].x);
            m.y = fmaf(p.ca, z[k].y, p.cb * x[k].y);
            m.z = fmaf(p.ca, z[k].z, p.cb * x[k].z);
            m.w = fmaf(p.ca, z[k].w, p.cb * x[k].w);
#pragma unroll
            for (int b = 0; b < FAN; ++b) {
                float4 c;
                if (WRITE) {
                    c.x = fmaf(p.g, xi[b].x, m.x);
                    c.y = fmaf(p.g, xi[b].y, m.y);
                    c.z = fmaf(p.g, xi[b].z, m.z);
                    c.w = fmaf(p.g, xi[b].w, m.w);
                    zc[static_cast<size_t>(b) * D4 + e] = c;
                } else {
                    c = __ldcs(zc + static_cast<size_t>(b) * D4 + e);
                }
                if (WRITE) {
                    // z' - mean is g xi up to the rounding of z' (relative 6e-8 of |z'|, far below the 1e-5 the log-prob
                    // is good to): sum xi^2 here, times g^2 once per warp below
                    acc[b] = fmaf(xi[b].x, xi[b].x, acc[b]);
                    acc[b] = fmaf(xi[b].y, xi[b].y, acc[b]);
                    acc[b] = fmaf(xi[b].z, xi[b].z, acc[b]);
                    acc[b] = fmaf(xi[b].w, xi[b].w, acc[b]);
                } else {
                    const float dx = c.x - m.x, dy = c.y - m.y, dz = c.z - m.z, dw = c.w - m.w;
                    acc[b] = fmaf(dx, dx, acc[b]);
                    acc[b] = fmaf(dy, dy, acc[b]);
                    acc[b] = fmaf(dz, dz, acc[b]);
                    acc[b] = fmaf(dw, dw, acc[b]);
                }
            }
        }
    }
}

template <int FAN, bool SHARED, bool WRITE, bool NOISY = true>
__global__ void __launch_bounds__(kStepThreads, kStepCtasPerSm)
step_kernel(const __grid_constant__ StepLaunch p) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    pdl_release();
    pdl_wait();           // the parents, the velocity and the pending partial sums come from earlier kernels
    // the previous level's log-probs (a handful of rows): summed by this launch
    if (p.prev.logp_out != nullptr)
        finalize_rows(p.prev, p.partialsf, p.n_trees, p.nodes_cap, p.nchunks, p.D, blockIdx.x * kStepWarps + warp, gridDim.x * kStepWarps, p.status, p.per_row);

    const int chunk = blockIdx.x % p.nchunks;
    const int row = blockIdx.x / p.nchunks;             // tree * W_in + j
    const int tree = row / p.W_in;
    const int j = row - tree * p.W_in;
    const uint32_t D4 = static_cast<uint32_t>(p.D >> 2);
    const uint32_t e_base = static_cast<uint32_t>(chunk) * kStepChunkVec;
    const uint32_t vecs = min(static_cast<uint32_t>(kStepChunkVec), D4 - e_base);
    const int64_t tree_row0 = static_cast<int64_t>(tree) * p.nodes_cap;
    const int parent = p.off_in + j;
    const int child0 = p.off_out + j * FAN;
    const bool streamed = (p.v != nullptr);
    if (!BGRPO_IN_BOUNDS(p.status, tree < p.n_trees && parent < p.nodes_cap && child0 + FAN <= p.nodes_cap && e_base < D4 &&
                                       (chunk + 1) * kStepWarps <= p.per_row)) return;
    const float4* __restrict__ zp = reinterpret_cast<const float4*>(p.latents + (tree_row0 + parent) * p.D) + e_base;
    const float4* __restrict__ xop = (streamed ? reinterpret_cast<const float4*>(p.v + static_cast<int64_t>(row) * p.D)
                                               : reinterpret_cast<const float4*>(p.mu + static_cast<int64_t>(tree) * p.D)) + e_base;
    float4* zc = reinterpret_cast<float4*>(p.latents + (tree_row0 + child0) * p.D);
    const uint32_t gid_parent = p.node_id_base + static_cast<uint32_t>(tree_row0 + parent);
    const uint32_t gid_child0 = p.node_id_base + static_cast<uint32_t>(tree_row0 + child0);

    float acc[FAN];
#pragma unroll
    for (int b = 0; b < FAN; ++b) acc[b] = 0.0f;
    float4 z[kStepVec], x[kStepVec];
    if (vecs == kStepChunkVec) {
        load_tile<true>(zp, xop, streamed, vecs, z, x);
        compute_tile<FAN, SHARED, WRITE, true, NOISY>(p, z, x, vecs, e_base, D4, zc, gid_parent, gid_child0, acc);
    } else {
        load_tile<false>(zp, xop, streamed, vecs, z, x);
        compute_tile<FAN, SHARED, WRITE, false, NOISY>(p, z, x, vecs, e_base, D4, zc, gid_parent, gid_child0, acc);
    }
    // one float per (child row, chunk, warp); summed later in a fixed order
#pragma unroll
    for (int b = 0; b < FAN; ++b) {
        float f = acc[b];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) f += __shfl_down_sync(0xffffffffu, f, o);
        if (WRITE) f *= p.g * p.g;
        if (lane == 0)
            p.partialsf[((tree_row0 + child0 + b) * p.nchunks + chunk) * kStepWarps + warp] = f;
    }
    if (WRITE && chunk == 0 && threadIdx.x < FAN) {      // node-table rows of the new children
        const int b = threadIdx.x;
        const int64_t rows = static_cast<int64_t>(p.n_trees) * p.nodes_cap;
        const int64_t r = tree_row0 + child0 + b, rp = tree_row0 + parent;
        p.table[r] = parent;
        p.table[rows + r] = p.step + 1;
        p.table[2 * rows + r] = p.is_split ? p.step : p.table[2 * rows + rp];
        p.table[3 * rows + r] = p.is_split ? b : p.table[3 * rows + rp];
    }
}

// Flush: adds up a pending level outside a step launch (the tree is complete, or tree_logprob is done).
__global__ void __launch_bounds__(kStreamThreads)
finalize_kernel(const FinalizeDesc f, const float* partialsf, int32_t n_trees, int32_t nodes_cap, int32_t nchunks, int64_t D,
                int32_t* status, int32_t per_row_cap) {
    pdl_release();
    pdl_wait();
    finalize_rows(f, partialsf, n_trees, nodes_cap, nchunks, D, blockIdx.x * (kStreamThreads / 32) + (threadIdx.x >> 5),
                  gridDim.x * (kStreamThreads / 32), status, per_row_cap);
}

__global__ void philox_words_kernel(const __grid_constant__ PhiloxKeys keys, uint32_t node, uint32_t step, uint32_t tag, uint4* out, int64_t nblk) {
    const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i < nblk) out[i] = philox4x32_10(make_uint4(static_cast<uint32_t>(i), node, step, tag), keys);
}
__global__ void philox_normals_kernel(const __grid_constant__ PhiloxKeys keys, uint32_t node, uint32_t step, uint32_t tag, float4* out, int64_t nblk) {
    const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i < nblk) out[i] = noise4(static_cast<uint32_t>(i), node, step, tag, keys);
}

__global__ void debug_trip_kernel(int32_t* status) {
    if (!BGRPO_IN_BOUNDS(status, threadIdx.x > 0)) return;      // thread 0 fails the test; nothing is accessed
}

template <int FAN>
cudaError_t launch_step_fan(const StepLaunch& p, unsigned int grid, cudaStream_t s) {
    if (!p.write_children) return launch_overlapped(step_kernel<FAN, false, false>, grid, kStepThreads, 0, s, p);
    if (p.g == 0.0f) return launch_overlapped(step_kernel<FAN, false, true, false>, grid, kStepThreads, 0, s, p);     // ODE step
    if (p.shared_noise) return launch_overlapped(step_kernel<FAN, true, true>, grid, kStepThreads, 0, s, p);
    return launch_overlapped(step_kernel<FAN, false, true>, grid, kStepThreads, 0, s, p);
}

}  // namespace

cudaError_t launch_debug_trip(int32_t* status, cudaStream_t s) {
    debug_trip_kernel<<<1, 32, 0, s>>>(status);
    return cudaGetLastError();
}

cudaError_t launch_root(const bgrpo_tree* t, cudaStream_t s) {
    const unsigned int grid = static_cast<unsigned int>(t->desc.n_trees) * t->nchunks;
    return launch_overlapped(root_kernel, grid, kStreamThreads, 0, s, t->buf.latents, t->buf.node_table, t->buf.logp, t->counters,
                             t->status, t->D, t->desc.n_trees, t->desc.nodes_cap, t->nchunks,
                             static_cast<uint32_t>(t->desc.tree_id_base * t->desc.nodes_cap), make_philox_keys(t->desc.seed));
}

cudaError_t launch_step(const StepLaunch& p, cudaStream_t s) {
    const int64_t items = static_cast<int64_t>(p.n_trees) * p.W_in * p.nchunks;
    if (items <= 0 || items > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
    const unsigned int grid = static_cast<unsigned int>(items);
    switch (p.fan) {
        case 1: return launch_step_fan<1>(p, grid, s);
        case 2: return launch_step_fan<2>(p, grid, s);
        case 3: return launch_step_fan<3>(p, grid, s);
        case 4: return launch_step_fan<4>(p, grid, s);
        default: return cudaErrorInvalidValue;
    }
}

cudaError_t launch_finalize(const bgrpo_tree* t, const FinalizeDesc& f, cudaStream_t s) {
    const int rows = t->desc.n_trees * f.W;
    const int grid = (rows + (kStreamThreads / 32) - 1) / (kStreamThreads / 32);
    return launch_overlapped(finalize_kernel, grid < 1 ? 1 : grid, kStreamThreads, 0, s, f, static_cast<const float*>(t->partialsf),
                             t->desc.n_trees, t->desc.nodes_cap, t->nchunks_step, t->D, t->status,
                             static_cast<int32_t>(partials_per_row(t->D)));
}

cudaError_t launch_philox_words(uint64_t seed, uint32_t node, uint32_t step, uint32_t tag, uint32_t* out, int64_t nblk, cudaStream_t s) {
    if (nblk <= 0) return cudaSuccess;
    philox_words_kernel<<<static_cast<unsigned int>((nblk + 255) / 256), 256, 0, s>>>(
        make_philox_keys(seed), node, step, tag, reinterpret_cast<uint4*>(out), nblk);
    return cudaGetLastError();
}
cudaError_t launch_philox_normals(uint64_t seed, uint32_t node, uint32_t step, uint32_t tag, float* out, int64_t n, cudaStream_t s) {
    if (n <= 0) return cudaSuccess;
    const int64_t nblk = n / 4;
    philox_normals_kernel<<<static_cast<unsigned int>((nblk + 255) / 256), 256, 0, s>>>(
        make_philox_keys(seed), node, step, tag, reinterpret_cast<float4*>(out), nblk);
    return cudaGetLastError();
}

}  // namespace bgrpo
