// Tree reductions: reward fusion (Eq. 3) + depth-wise normalisation (Eq. 4) in one kernel, and the width / depth
// pruning masks ("Pruning Strategies") in another.  A tree usually has at most a few thousand nodes, so one CTA owns one
// tree, keeps the per-node state in shared memory as doubles and walks the levels; the kernels are latency-bound.
// A tree whose per-node state does not fit in shared memory (more than about 8 500 nodes: K = 4 with seven splits, say)
// keeps it in the caller's scratch instead; the code is the same, only the pointer differs.
//
// Fusion uses the bottom-up form of Eq. 3.  With a_c = beta*logp(c) the softmax weight of leaf l under node n
// factorises along the path, so  S_n = sum_c e^{a_c} S_c,  R_n = sum_c e^{a_c} R_c,  rbar(n) = R_n / S_n  with
// S_leaf = 1, R_leaf = r.  S is carried as log S (shifted by the largest term) so huge |beta*logp| cannot overflow;
// R/S is carried directly as rbar:  rbar(n) = sum_c w_c rbar(c),  w_c = e^{a_c + logS_c - m} / sum_c' e^{a_c' + logS_c' - m}.
#include "internal.h"

namespace bgrpo {
namespace {

constexpr int kTreeThreads = 256;

__device__ __forceinline__ double warp_sum_d(double x) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}

__global__ void __launch_bounds__(kTreeThreads)
fuse_advantage_kernel(const FuseLaunch p) {
    pdl_release();
    pdl_wait();
    extern __shared__ double sm[];
    const int tree = blockIdx.x;
    const bool in_smem = static_cast<size_t>(p.nodes) * 3 * sizeof(double) <= kTreeSmemLimit;
    double* rb = in_smem ? sm : p.node_scratch + static_cast<int64_t>(tree) * 2 * p.nodes_cap;   // rbar per node
    double* ls = rb + (in_smem ? p.nodes : p.nodes_cap);                                          // log S per node
    double* la = in_smem ? ls + p.nodes : nullptr;     // beta * logp per node, fetched once (a level then waits for no global load)
    const int64_t row0 = static_cast<int64_t>(tree) * p.nodes_cap;
    const int T = p.T;
    const int leaves = p.lv.width[T];
    const int off_leaf = p.lv.offset[T];
    __shared__ int bad;
    if (threadIdx.x == 0) bad = 0;
    __syncthreads();
    const double beta = p.beta_scaled;
    if (la)
        for (int n = threadIdx.x; n < p.nodes; n += kTreeThreads) la[n] = beta * static_cast<double>(p.logp[row0 + n]);
    for (int l = threadIdx.x; l < leaves; l += kTreeThreads) {
        const float r = p.leaf_r[static_cast<int64_t>(tree) * leaves + l];
        if (!isfinite(r)) bad = 1;
        rb[off_leaf + l] = static_cast<double>(r);
        ls[off_leaf + l] = 0.0;
    }
    __syncthreads();
    if (bad && threadIdx.x == 0) atomicOr(p.status, 1);
    for (int d = T - 1; d >= 0; --d) {
        const int fan = p.lv.fanout[d];
        const int off = p.lv.offset[d], offc = p.lv.offset[d + 1];
        for (int j = threadIdx.x; j < p.lv.width[d]; j += kTreeThreads) {
            const int c0 = offc + j * fan;
            if (!BGRPO_IN_BOUNDS(p.status, off + j < offc && c0 + fan <= p.nodes && p.nodes <= p.nodes_cap)) continue;
            if (fan == 1) {      // an only child: its value is the parent's, and log S just picks up the edge
                rb[off + j] = rb[c0];
                ls[off + j] = (la ? la[c0] : beta * static_cast<double>(p.logp[row0 + c0])) + ls[c0];
                continue;
            }
            if (beta == 0.0) {   // uniform weights: every child of a node has the same number of leaves below it, so the
                                 // leaf mean of the parent is the plain mean of its children's leaf means
                double R = 0.0;
#pragma unroll
                for (int b = 0; b < BGRPO_MAX_K; ++b)
                    if (b < fan) R += rb[c0 + b];
                rb[off + j] = R / fan;
                ls[off + j] = 0.0;
                continue;
            }
            double a[BGRPO_MAX_K];
            double m = -INFINITY;
#pragma unroll
            for (int b = 0; b < BGRPO_MAX_K; ++b) {
                if (b < fan) {
                    a[b] = (la ? la[c0 + b] : beta * static_cast<double>(p.logp[row0 + c0 + b])) + ls[c0 + b];
                    m = fmax(m, a[b]);
                }
            }
            double S = 0.0, R = 0.0;
#pragma unroll
            for (int b = 0; b < BGRPO_MAX_K; ++b) {
                if (b < fan) {
                    const double w = exp(a[b] - m);
                    S += w;
                    R += w * rb[c0 + b];
                }
            }
            rb[off + j] = R / S;
            ls[off + j] = m + log(S);
        }
        __syncthreads();
    }
    // Depth-wise statistics: one warp per depth, two passes (mean, then centred squares), fixed lane order.
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int d = warp; d <= T; d += kTreeThreads / 32) {
        const int W = p.lv.width[d], off = p.lv.offset[d];
        double s = 0.0;
        for (int j = lane; j < W; j += 32) s += rb[off + j];
        const double mean = warp_sum_d(s) / W;
        double q = 0.0;
        for (int j = lane; j < W; j += 32) { const double c = rb[off + j] - mean; q += c * c; }
        const double sd = sqrt(warp_sum_d(q) / W);
        const double inv = 1.0 / (sd + static_cast<double>(p.eps));
        for (int j = lane; j < W; j += 32) {
            double A = (d == 0) ? 0.0 : (rb[off + j] - mean) * inv;
            if (p.clip > 0.0f) A = fmin(fmax(A, -static_cast<double>(p.clip)), static_cast<double>(p.clip));
            p.adv[row0 + off + j] = static_cast<float>(A);
            p.rbar[row0 + off + j] = static_cast<float>(rb[off + j]);
        }
    }
}

// Effective sample size of the fusion weights (appendix "Reward Fusion"): ESS(n) = (sum_l w_l)^2 / sum_l w_l^2 over the
// descendant leaves of n, w_l = exp(beta s_l).  Both sums factorise along the paths like S above:
//   log S_n = logsumexp_c(a_c + log S_c),   log Q_n = logsumexp_c(2 a_c + log Q_c),   ESS = exp(2 log S - log Q).
__global__ void __launch_bounds__(kTreeThreads)
fusion_ess_kernel(const EssLaunch p) {
    pdl_release();
    pdl_wait();
    extern __shared__ double sm[];
    const int tree = blockIdx.x;
    const bool in_smem = static_cast<size_t>(p.nodes) * 2 * sizeof(double) <= kTreeSmemLimit;
    double* ls = in_smem ? sm : p.node_scratch + static_cast<int64_t>(tree) * 2 * p.nodes_cap;
    double* lq = ls + (in_smem ? p.nodes : p.nodes_cap);
    const int64_t row0 = static_cast<int64_t>(tree) * p.nodes_cap;
    const int T = p.T;
    for (int l = threadIdx.x; l < p.lv.width[T]; l += kTreeThreads) {
        ls[p.lv.offset[T] + l] = 0.0;
        lq[p.lv.offset[T] + l] = 0.0;
        p.ess[row0 + p.lv.offset[T] + l] = 1.0f;
    }
    __syncthreads();
    for (int d = T - 1; d >= 0; --d) {
        const int fan = p.lv.fanout[d];
        const int off = p.lv.offset[d], offc = p.lv.offset[d + 1];
        for (int j = threadIdx.x; j < p.lv.width[d]; j += kTreeThreads) {
            const int c0 = offc + j * fan;
            if (!BGRPO_IN_BOUNDS(p.status, off + j < offc && c0 + fan <= p.nodes && p.nodes <= p.nodes_cap)) continue;
            double a1[BGRPO_MAX_K], a2[BGRPO_MAX_K];
            double m1 = -INFINITY, m2 = -INFINITY;
#pragma unroll
            for (int b = 0; b < BGRPO_MAX_K; ++b) {
                if (b < fan) {
                    const double a = p.beta_scaled * static_cast<double>(p.logp[row0 + c0 + b]);
                    a1[b] = a + ls[c0 + b];
                    a2[b] = 2.0 * a + lq[c0 + b];
                    m1 = fmax(m1, a1[b]);
                    m2 = fmax(m2, a2[b]);
                }
            }
            double S = 0.0, Q = 0.0;
#pragma unroll
            for (int b = 0; b < BGRPO_MAX_K; ++b) {
                if (b < fan) {
                    S += exp(a1[b] - m1);
                    Q += exp(a2[b] - m2);
                }
            }
            const double lS = m1 + log(S), lQ = m2 + log(Q);
            ls[off + j] = lS;
            lq[off + j] = lQ;
            p.ess[row0 + off + j] = static_cast<float>(exp(2.0 * lS - lQ));
        }
        __syncthreads();
    }
}

// rank of x among its siblings: number of entries that beat it (larger value, or equal value and lower index)
__device__ __forceinline__ bool beats(float v_other, int i_other, float v_me, int i_me) {
    return (v_other > v_me) || (v_other == v_me && i_other < i_me);
}

// Sort keys of the Extreme-b selection.  A float32 maps to an unsigned integer of the same order (sign bit flipped for
// non-negative values, all bits for negative ones); the leaf index goes below it, complemented, so that among equal
// values the lower index has the larger key.  "best" ranks large values first, "worst" small values first: the b
// leaves with the largest keys are the ones the ranking "value, ties to the lower leaf index" puts first.
__device__ __forceinline__ uint64_t extreme_key(float v, uint32_t leaf, bool worst) {
    uint32_t u = __float_as_uint(v);
    if ((u << 1) == 0u) u = 0u;                              // -0 and +0 compare equal
    u = (u & 0x80000000u) ? ~u : (u | 0x80000000u);
    if (worst) u = ~u;
    return (static_cast<uint64_t>(u) << 32) | static_cast<uint64_t>(~leaf);
}

// The want-th largest key among the tree's leaves (1 <= want <= L): radix selection, eight passes of eight bits over
// the 64-bit keys; every pass histograms the keys that share the prefix fixed so far.  Keys are distinct (they hold
// the leaf index), so exactly `want` leaves have a key >= the result.  Called by the whole CTA.
__device__ uint64_t select_kth_largest(const float* leaf_vals, int L, int want, bool worst, unsigned int* hist, uint64_t* shared_prefix,
                                       int* shared_want) {
    if (threadIdx.x == 0) { *shared_prefix = 0; *shared_want = want; }
    for (int pass = 7; pass >= 0; --pass) {
        for (int i = threadIdx.x; i < 256; i += kTreeThreads) hist[i] = 0u;
        __syncthreads();
        const uint64_t prefix = *shared_prefix;
        const int shift = 8 * pass;
        for (int l = threadIdx.x; l < L; l += kTreeThreads) {
            const uint64_t key = extreme_key(leaf_vals[l], static_cast<uint32_t>(l), worst);
            const bool same_prefix = (pass == 7) || ((key >> (shift + 8)) == (prefix >> (shift + 8)));
            if (same_prefix) atomicAdd(&hist[static_cast<unsigned int>(key >> shift) & 255u], 1u);
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            int left = *shared_want, bin = 255;
            for (; bin > 0; --bin) {                        // bins from the largest digit down
                const int c = static_cast<int>(hist[bin]);
                if (c >= left) break;
                left -= c;
            }
            *shared_want = left;
            *shared_prefix = prefix | (static_cast<uint64_t>(bin) << shift);
        }
        __syncthreads();
    }
    return *shared_prefix;
}

__global__ void __launch_bounds__(kTreeThreads)
prune_kernel(const PruneLaunch p) {
    pdl_release();
    pdl_wait();
    extern __shared__ unsigned char prune_smem[];      // small trees: the node values as floats
    const int tree = blockIdx.x;
    const int64_t row0 = static_cast<int64_t>(tree) * p.nodes_cap;
    const int T = p.T;
    const float* rbar = p.rbar + row0;
    if (p.values_in_smem) {        // fetched once: a level then waits for no global load
        float* vals = reinterpret_cast<float*>(prune_smem);
        for (int n = threadIdx.x; n < p.nodes; n += kTreeThreads) vals[n] = rbar[n];
        rbar = vals;
        __syncthreads();
    }
    if (p.mode == BGRPO_WIDTH_EXTREME_B) {
        // The mask itself holds the keep flags while they are gathered: 0 everywhere, 1 on the root paths of the
        // selected leaves (several threads may write the same 1), then the depth conditions are applied in place.
        __shared__ unsigned int hist[256];
        __shared__ uint64_t s_prefix;
        __shared__ int s_want;
        uint8_t* keep = p.mask + row0;
        for (int n = threadIdx.x; n < p.nodes; n += kTreeThreads) keep[n] = 0;
        const int L = p.lv.width[T], off = p.lv.offset[T];
        const int want = p.k < L ? p.k : L;
        const uint64_t best_cut = select_kth_largest(rbar + off, L, want, false, hist, &s_prefix, &s_want);
        __syncthreads();
        const uint64_t worst_cut = select_kth_largest(rbar + off, L, want, true, hist, &s_prefix, &s_want);
        __syncthreads();                                   // also orders the zero fill before the flags below
        for (int l = threadIdx.x; l < L; l += kTreeThreads) {
            const float v = rbar[off + l];
            if (extreme_key(v, static_cast<uint32_t>(l), false) >= best_cut || extreme_key(v, static_cast<uint32_t>(l), true) >= worst_cut) {
                int n = off + l;
                for (int guard = 0; n >= 0 && guard <= T; ++guard) {       // root path through the node table
                    if (!BGRPO_IN_BOUNDS(p.status, n < p.nodes)) break;
                    keep[n] = 1;
                    n = p.table[row0 + n];
                }
            }
        }
        __syncthreads();
        for (int d = 0; d <= T; ++d) {
            const bool depth_ok = d > 0 && !((p.pruned_bits >> (d - 1)) & 1ull) && !(p.ignore_last && d == T);
            const int offd = p.lv.offset[d];
            for (int j = threadIdx.x; j < p.lv.width[d]; j += kTreeThreads)
                if (!depth_ok) keep[offd + j] = 0;
        }
        return;
    }
    // Top-k modes: a node is kept iff, at every ranked split on its root path, the ancestor (or the node itself)
    // ranks among the k best of its siblings.  Every node walks its own path (children of the j-th node of depth d
    // are j*F + b of depth d+1, so the parent of j is j / F): no level-by-level pass, no barrier.
    __shared__ int s_off[BGRPO_MAX_T + 2], s_fan[BGRPO_MAX_T];
    for (int i = threadIdx.x; i <= T + 1; i += kTreeThreads) s_off[i] = p.lv.offset[i];
    for (int i = threadIdx.x; i < T; i += kTreeThreads) s_fan[i] = p.lv.fanout[i];
    __syncthreads();
    for (int n = threadIdx.x; n < p.nodes; n += kTreeThreads) {       // one node per thread, all depths at once
        int d = 0;
        while (d < T && n >= s_off[d + 1]) ++d;
        const bool depth_ok = d > 0 && !((p.pruned_bits >> (d - 1)) & 1ull) && !(p.ignore_last && d == T);
        bool kept = true;
        int j = n - s_off[d];
        for (int e = d; e > 0 && kept; --e) {                // e: depth of the node j on the path
            const int fan = s_fan[e - 1];
            const int pj = j / fan, b = j - pj * fan;
            const bool ranked = fan > 1 && (p.mode == BGRPO_WIDTH_PER_SPLIT_TOPK ||
                                            (p.mode == BGRPO_WIDTH_LAST_SPLIT_TOPK && e - 1 == p.last_split));
            if (ranked) {
                const int sib0 = s_off[e] + pj * fan;
                if (!BGRPO_IN_BOUNDS(p.status, sib0 >= 0 && sib0 + fan <= p.nodes)) break;
                const float v = rbar[sib0 + b];
                int rank = 0;
                for (int q = 0; q < fan; ++q) rank += beats(rbar[sib0 + q], q, v, b) ? 1 : 0;
                kept = rank < p.k;
            }
            j = pj;
        }
        p.mask[row0 + n] = (depth_ok && kept) ? 1 : 0;
    }
}

// Clipped GRPO objective (Eq. 5), forward value: one CTA per tree; per-thread strided sums, fixed-order reduction.
__global__ void __launch_bounds__(kTreeThreads)
objective_kernel(const ObjectiveLaunch p) {
    pdl_release();
    pdl_wait();
    const int tree = blockIdx.x;
    const int64_t row0 = static_cast<int64_t>(tree) * p.nodes_cap;
    double sum = 0.0;
    int cnt = 0;
    if (!BGRPO_IN_BOUNDS(p.status, p.nodes <= p.nodes_cap && tree < p.n_trees)) return;
    for (int n = threadIdx.x; n < p.nodes; n += kTreeThreads) {
        float term = 0.0f;
        if (n > 0 && p.mask[row0 + n]) {
            const double rho = exp(p.logp_scale * (static_cast<double>(p.logp_new[row0 + n]) - static_cast<double>(p.logp_old[row0 + n])));
            const double a = static_cast<double>(p.adv[row0 + n]);
            const double lo = 1.0 - static_cast<double>(p.clip_eps), hi = 1.0 + static_cast<double>(p.clip_eps);
            const double t = fmin(rho * a, fmin(fmax(rho, lo), hi) * a);
            sum += t;
            cnt += 1;
            term = static_cast<float>(t);
        }
        if (p.terms) p.terms[row0 + n] = term;
    }
    __shared__ double ssum[kTreeThreads / 32];
    __shared__ int scnt[kTreeThreads / 32];
    sum = warp_sum_d(sum);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
    if ((threadIdx.x & 31) == 0) { ssum[threadIdx.x >> 5] = sum; scnt[threadIdx.x >> 5] = cnt; }
    __syncthreads();
    if (threadIdx.x == 0) {
        double s = 0.0;
        int c = 0;
        for (int w = 0; w < kTreeThreads / 32; ++w) { s += ssum[w]; c += scnt[w]; }
        p.J[tree] = c > 0 ? static_cast<float>(s / c) : 0.0f;
    }
}

}  // namespace

cudaError_t launch_objective(const ObjectiveLaunch& p, cudaStream_t s) {
    return launch_overlapped(objective_kernel, p.n_trees, kTreeThreads, 0, s, p);
}

cudaError_t launch_fusion_ess(const EssLaunch& p, cudaStream_t s) {
    size_t smem = static_cast<size_t>(p.nodes) * 2 * sizeof(double);
    if (smem > kTreeSmemLimit) smem = 0;          // per-node state in the caller's scratch
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(fusion_ess_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
        if (e != cudaSuccess) return e;
    }
    return launch_overlapped(fusion_ess_kernel, p.n_trees, kTreeThreads, smem, s, p);
}

cudaError_t launch_fuse_advantage(const FuseLaunch& p, cudaStream_t s) {
    size_t smem = static_cast<size_t>(p.nodes) * 3 * sizeof(double);
    if (smem > kTreeSmemLimit) smem = 0;          // per-node state in the caller's scratch
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(fuse_advantage_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
        if (e != cudaSuccess) return e;
    }
    return launch_overlapped(fuse_advantage_kernel, p.n_trees, kTreeThreads, smem, s, p);
}

cudaError_t launch_prune(const PruneLaunch& p0, cudaStream_t s) {
    PruneLaunch p = p0;
    size_t smem = static_cast<size_t>(p.nodes) * sizeof(float);
    p.values_in_smem = smem <= kTreeSmemLimit ? 1 : 0;       // larger trees read the values from global memory
    if (!p.values_in_smem) smem = 0;
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(prune_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
        if (e != cudaSuccess) return e;
    }
    return launch_overlapped(prune_kernel, p.n_trees, kTreeThreads, smem, s, p);
}

}  // namespace bgrpo
