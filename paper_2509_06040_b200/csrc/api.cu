// C ABI of the library: argument checks, the host mirror of the tree layout, per-step coefficients and launches.
// No device memory is allocated here; every kernel is enqueued on the caller's stream.
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>

#include "internal.h"

using namespace bgrpo;

namespace {

thread_local char g_last_error[256] = "";

bgrpo_status cuda_fail(cudaError_t e, const char* where) {
    snprintf(g_last_error, sizeof(g_last_error), "%s: %s", where, cudaGetErrorString(e));
    return BGRPO_ERR_CUDA;
}
bgrpo_status fail(bgrpo_status s, const char* why) {
    snprintf(g_last_error, sizeof(g_last_error), "%s", why);
    return s;
}

inline cudaStream_t as_stream(void* s) { return static_cast<cudaStream_t>(s); }
inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

bgrpo_status check_desc(const bgrpo_tree_desc* d) {
    if (!d) return fail(BGRPO_ERR_INVALID_ARG, "desc is NULL");
    if (d->n_trees < 1 || d->tokens < 1 || d->channels < 1) return fail(BGRPO_ERR_INVALID_ARG, "n_trees, tokens, channels must be >= 1");
    const int64_t D = static_cast<int64_t>(d->tokens) * d->channels;
    if (D % 4 != 0) return fail(BGRPO_ERR_INVALID_ARG, "tokens*channels must be a multiple of 4");
    if (D / 4 > 0x7fffffffLL) return fail(BGRPO_ERR_INVALID_ARG, "row too long for the 32-bit block counter");
    if (d->T < 1 || d->T > BGRPO_MAX_T) return fail(BGRPO_ERR_INVALID_ARG, "T out of range");
    if (d->K < 1 || d->K > BGRPO_MAX_K) return fail(BGRPO_ERR_INVALID_ARG, "K out of range");
    if (d->nodes_cap < d->T + 1) return fail(BGRPO_ERR_INVALID_ARG, "nodes_cap smaller than a split-free tree");
    if (d->tree_id_base < 0) return fail(BGRPO_ERR_INVALID_ARG, "tree_id_base negative");
    if (!(d->sigma >= 0.0f) || !std::isfinite(d->sigma)) return fail(BGRPO_ERR_INVALID_ARG, "sigma must be finite and >= 0");
    if (std::isnan(d->branch_corr_s)) return fail(BGRPO_ERR_INVALID_ARG, "branch_corr_s is NaN");
    return BGRPO_OK;
}

int nchunks_of(int64_t D) { return static_cast<int>((D / 4 + kChunkVec - 1) / kChunkVec); }
int nchunks_step_of(int64_t D) { return static_cast<int>((D / 4 + kStepChunkVec - 1) / kStepChunkVec); }

size_t scratch_bytes_of(const bgrpo_tree_desc* d) {
    const int64_t rows = static_cast<int64_t>(d->n_trees) * d->nodes_cap;
    const int64_t D = static_cast<int64_t>(d->tokens) * d->channels;
    size_t b = kScratchHeader;
    b += ((static_cast<size_t>(rows) * sizeof(unsigned int) + 255) / 256) * 256;
    b += static_cast<size_t>(rows) * nchunks_of(D) * 3 * sizeof(double);
    b += static_cast<size_t>(rows) * 2 * sizeof(double);
    b += static_cast<size_t>(rows) * static_cast<size_t>(partials_per_row(D)) * sizeof(float);
    if (d->channels == BGRPO_MLP_CHANNELS) b = ((b + 255) / 256) * 256 + kMlpTicketBytes + kMlpPartialBytes;
    return b;
}

void fill_coefficients(bgrpo_tree* t) {
    for (int i = 0; i < t->desc.T; ++i) {
        const double sigma = ((t->ode_bits >> i) & 1ull) ? 0.0 : static_cast<double>(t->desc.sigma);   // ODE steps of the hybrid schedule
        const double ti = t->t_grid[i], h = static_cast<double>(t->t_grid[i]) - static_cast<double>(t->t_grid[i + 1]);
        const double c = sigma * sigma * h / (2.0 * ti);
        const double a = 1.0 - c, b = -(h + c * (1.0 - ti));
        StepCoef& k = t->coef[i];
        k.a = static_cast<float>(a);
        k.b = static_cast<float>(b);
        const double g = sigma * std::sqrt(h);
        k.g = static_cast<float>(g);
        k.inv_2g2 = g > 0 ? static_cast<float>(1.0 / (2.0 * g * g)) : 0.0f;
        k.logp_const = g > 0 ? static_cast<float>(-std::log(g) - 0.5 * std::log(2.0 * M_PI)) : 0.0f;
        if (t->mu) {
            const double s0 = t->s0;
            const double ct = (1.0 - ti) * (1.0 - ti) * s0 * s0 + ti * ti;
            const double kt = (ti - (1.0 - ti) * s0 * s0) / ct;
            // v = kt z - (1 + kt (1-t)) mu  =>  mean = (a + b kt) z - b (1 + kt (1-t)) mu
            k.lin_a = static_cast<float>(a + b * kt);
            k.lin_b = static_cast<float>(-b * (1.0 + kt * (1.0 - ti)));
        } else {
            k.lin_a = k.lin_b = 0.0f;
        }
    }
}

// Everything of the handle that follows from the description and the buffers alone: sizes, noise mixing, the carving of
// the scratch allocation.  No velocity bound, every step stochastic, nothing pending.
void bind_buffers(bgrpo_tree* t, const bgrpo_buffers* b) {
    const bgrpo_tree_desc* desc = &t->desc;
    t->buf = *b;
    t->D = static_cast<int64_t>(desc->tokens) * desc->channels;
    t->nchunks = nchunks_of(t->D);
    t->nchunks_step = nchunks_step_of(t->D);
    t->nchunks_reward = static_cast<int32_t>((t->D / 4 + kRewardChunkVec - 1) / kRewardChunkVec);
    t->independent = !(std::isfinite(desc->branch_corr_s) && desc->branch_corr_s >= 0.0f);
    if (t->independent) {
        t->mix_shared = 0.0f;
        t->mix_innov = 1.0f;
    } else {
        const double s = desc->branch_corr_s, n = std::sqrt(1.0 + s * s);
        t->mix_shared = static_cast<float>(1.0 / n);
        t->mix_innov = static_cast<float>(s / n);
    }
    t->mu = nullptr;
    t->s0 = 0.0f;
    t->ode_bits = 0;
    char* sc = static_cast<char*>(b->scratch);
    const size_t rows = static_cast<size_t>(desc->n_trees) * desc->nodes_cap;
    t->status = reinterpret_cast<int32_t*>(sc);
    t->counters = reinterpret_cast<unsigned int*>(sc + kScratchHeader);
    t->partials = reinterpret_cast<double*>(sc + kScratchHeader + ((rows * sizeof(unsigned int) + 255) / 256) * 256);
    t->node_scratch = t->partials + rows * static_cast<size_t>(t->nchunks) * 3;
    t->partialsf = reinterpret_cast<float*>(t->node_scratch + rows * 2);
    t->mlp_tickets = nullptr;
    t->mlp_partials = nullptr;
    if (desc->channels == BGRPO_MLP_CHANNELS) {
        const size_t used = reinterpret_cast<char*>(t->partialsf + rows * static_cast<size_t>(partials_per_row(t->D))) - sc;
        t->mlp_tickets = reinterpret_cast<unsigned int*>(sc + ((used + 255) / 256) * 256);
        t->mlp_partials = reinterpret_cast<float*>(reinterpret_cast<char*>(t->mlp_tickets) + kMlpTicketBytes);
    }
    t->pending.logp_out = nullptr;
}

bool tree_complete(const bgrpo_tree* t) { return t->depth == t->desc.T; }

// Enqueues the small kernel that adds up a level's pending log-prob partials, if there are any.
cudaError_t flush_pending(bgrpo_tree* t, cudaStream_t s) {
    if (!t->pending.logp_out) return cudaSuccess;
    const cudaError_t e = launch_finalize(t, t->pending, s);
    t->pending.logp_out = nullptr;
    return e;
}

}  // namespace

extern "C" {

const char* bgrpo_status_string(bgrpo_status s) {
    switch (s) {
        case BGRPO_OK: return "ok";
        case BGRPO_ERR_INVALID_ARG: return "invalid argument";
        case BGRPO_ERR_STATE: return "call out of order for the tree's state";
        case BGRPO_ERR_CAPACITY: return "capacity exceeded";
        case BGRPO_ERR_NONFINITE: return "non-finite value met on the device";
        case BGRPO_ERR_CUDA: return "CUDA error";
        case BGRPO_ERR_UNSUPPORTED: return "unsupported";
    }
    return "unknown status";
}

const char* bgrpo_last_error(void) { return g_last_error; }

bgrpo_status bgrpo_tree_workspace(const bgrpo_tree_desc* desc, bgrpo_sizes* out) {
    if (!out) return fail(BGRPO_ERR_INVALID_ARG, "out is NULL");
    bgrpo_status st = check_desc(desc);
    if (st != BGRPO_OK) return st;
    const size_t rows = static_cast<size_t>(desc->n_trees) * desc->nodes_cap;
    const size_t D = static_cast<size_t>(desc->tokens) * desc->channels;
    out->latents_bytes = rows * D * sizeof(float);
    out->node_table_bytes = 4 * rows * sizeof(int32_t);
    out->per_node_float_bytes = rows * sizeof(float);
    out->mask_bytes = rows;
    out->scratch_bytes = scratch_bytes_of(desc);
    return BGRPO_OK;
}

bgrpo_status bgrpo_tree_count(int32_t T, int32_t K, const int32_t* split_steps, int32_t n_splits, int64_t* nodes,
                              int64_t* node_steps, int64_t* model_evals, int64_t* leaves) {
    if (T < 1 || T > BGRPO_MAX_T || K < 1 || K > BGRPO_MAX_K || n_splits < 0 || n_splits > T || (n_splits > 0 && !split_steps))
        return fail(BGRPO_ERR_INVALID_ARG, "bad schedule");
    bool is_split[BGRPO_MAX_T] = {false};
    for (int q = 0; q < n_splits; ++q) {
        if (split_steps[q] < 0 || split_steps[q] >= T || is_split[split_steps[q]]) return fail(BGRPO_ERR_INVALID_ARG, "split steps must be distinct and in 0..T-1");
        is_split[split_steps[q]] = true;
    }
    int64_t w = 1, total = 1;
    for (int i = 0; i < T; ++i) {
        if (is_split[i]) w *= K;
        if (w > (1LL << 40)) return fail(BGRPO_ERR_CAPACITY, "tree too wide");
        total += w;
    }
    if (nodes) *nodes = total;
    if (node_steps) *node_steps = total - 1;
    if (model_evals) *model_evals = total - w;
    if (leaves) *leaves = w;
    return BGRPO_OK;
}

bgrpo_status bgrpo_tree_init(const bgrpo_tree_desc* desc, const bgrpo_buffers* b, void* stream, bgrpo_tree** out) {
    if (!out) return fail(BGRPO_ERR_INVALID_ARG, "out is NULL");
    bgrpo_status st = check_desc(desc);
    if (st != BGRPO_OK) return st;
    if (!b || !b->latents || !b->node_table || !b->logp || !b->rbar || !b->adv || !b->mask || !b->scratch)
        return fail(BGRPO_ERR_INVALID_ARG, "a device buffer is NULL");
    if (!desc->t_grid) return fail(BGRPO_ERR_INVALID_ARG, "t_grid is NULL");
    if (!aligned(b->latents, 16) || !aligned(b->scratch, 256) || !aligned(b->node_table, 4) || !aligned(b->logp, 4))
        return fail(BGRPO_ERR_INVALID_ARG, "misaligned device buffer");
    for (int i = 0; i <= desc->T; ++i) {
        const float t = desc->t_grid[i];
        if (!std::isfinite(t) || t > 1.0f || t < 0.0f) return fail(BGRPO_ERR_INVALID_ARG, "t_grid values must lie in [0, 1]");
        if (i > 0 && !(t < desc->t_grid[i - 1])) return fail(BGRPO_ERR_INVALID_ARG, "t_grid must be strictly decreasing");
    }
    if (!(desc->t_grid[desc->T - 1] > 0.0f)) return fail(BGRPO_ERR_INVALID_ARG, "t_grid[T-1] must be > 0");
    if (b->scratch_bytes < scratch_bytes_of(desc)) return fail(BGRPO_ERR_CAPACITY, "scratch_bytes too small");
    const int64_t last_id = (desc->tree_id_base + desc->n_trees) * static_cast<int64_t>(desc->nodes_cap);
    if (last_id > 0xffffffffLL) return fail(BGRPO_ERR_CAPACITY, "global node ids exceed 32 bits");

    bgrpo_tree* t = new (std::nothrow) bgrpo_tree();
    if (!t) return fail(BGRPO_ERR_INVALID_ARG, "out of host memory");
    t->desc = *desc;
    std::memcpy(t->t_grid, desc->t_grid, sizeof(float) * (desc->T + 1));
    t->desc.t_grid = t->t_grid;
    bind_buffers(t, b);
    fill_coefficients(t);
    st = bgrpo_tree_reset(t, desc->seed, stream);
    if (st == BGRPO_OK && t->mlp_tickets) {      // the MLP stage's tile tickets start at zero and return to zero after every launch
        const cudaError_t e = cudaMemsetAsync(t->mlp_tickets, 0, kMlpTicketBytes, as_stream(stream));
        if (e != cudaSuccess) st = cuda_fail(e, "clearing the MLP tickets");
    }
    if (st != BGRPO_OK) {
        delete t;
        return st;
    }
    *out = t;
    return BGRPO_OK;
}

bgrpo_status bgrpo_tree_reset(bgrpo_tree* t, uint64_t seed, void* stream) {
    if (!t) return fail(BGRPO_ERR_INVALID_ARG, "tree is NULL");
    t->desc.seed = seed;
    t->pending.logp_out = nullptr;
    t->depth = 0;
    std::memset(&t->lv, 0, sizeof(t->lv));
    t->lv.width[0] = 1;
    t->lv.offset[0] = 0;
    t->lv.offset[1] = 1;
    cudaError_t e = launch_root(t, as_stream(stream));
    if (e != cudaSuccess) return cuda_fail(e, "root kernel");

    return BGRPO_OK;
}

bgrpo_status bgrpo_velocity_linear_bind(bgrpo_tree* t, const float* mu_dev, float s0) {
    if (!t || !mu_dev) return fail(BGRPO_ERR_INVALID_ARG, "tree or mu is NULL");
    if (!(s0 > 0.0f) || !std::isfinite(s0)) return fail(BGRPO_ERR_INVALID_ARG, "s0 must be finite and > 0");
    if (!aligned(mu_dev, 16)) return fail(BGRPO_ERR_INVALID_ARG, "mu misaligned");
    t->mu = mu_dev;
    t->s0 = s0;
    fill_coefficients(t);
    return BGRPO_OK;
}

static void fill_step_launch(const bgrpo_tree* t, int step, const float* v_dev, StepLaunch* p) {
    const StepCoef& k = t->coef[step];
    p->latents = t->buf.latents;
    p->v = v_dev;
    p->mu = v_dev ? nullptr : t->mu;
    p->logp = t->buf.logp;
    p->table = t->buf.node_table;
    p->partialsf = t->partialsf;
    p->status = t->status;
    p->per_row = static_cast<int32_t>(partials_per_row(t->D));
    p->prev = t->pending;
    p->D = t->D;
    p->n_trees = t->desc.n_trees;
    p->nodes_cap = t->desc.nodes_cap;
    p->nchunks = t->nchunks_step;
    p->step = step;
    p->node_id_base = static_cast<uint32_t>(t->desc.tree_id_base * t->desc.nodes_cap);
    p->keys = make_philox_keys(t->desc.seed);
    p->ca = v_dev ? k.a : k.lin_a;
    p->cb = v_dev ? k.b : k.lin_b;
    p->g = k.g;
    p->inv_2g2 = k.inv_2g2;
    p->logp_const = k.logp_const;
    p->mix_shared = t->mix_shared;
    p->mix_innov = t->mix_innov;
}

bgrpo_status bgrpo_tree_step(bgrpo_tree* t, int32_t split_flag, const float* v_dev, void* stream) {
    if (!t) return fail(BGRPO_ERR_INVALID_ARG, "tree is NULL");
    if (t->depth >= t->desc.T) return fail(BGRPO_ERR_STATE, "tree already at depth T");
    if (!v_dev && !t->mu) return fail(BGRPO_ERR_STATE, "no velocity: pass v_dev or bind a linear velocity");
    if (v_dev && !aligned(v_dev, 16)) return fail(BGRPO_ERR_INVALID_ARG, "v misaligned");
    const int i = t->depth;
    if (split_flag && ((t->ode_bits >> i) & 1ull) && t->desc.sigma > 0.0f)
        return fail(BGRPO_ERR_INVALID_ARG, "a split step must be an SDE step of the hybrid schedule");
    const int fan = split_flag ? t->desc.K : 1;
    const int64_t W_out = static_cast<int64_t>(t->lv.width[i]) * fan;
    const int64_t off_out = t->lv.offset[i + 1];
    if (off_out + W_out > t->desc.nodes_cap) return fail(BGRPO_ERR_CAPACITY, "children exceed nodes_cap");
    StepLaunch p;
    fill_step_launch(t, i, v_dev, &p);
    p.W_in = t->lv.width[i];
    p.off_in = t->lv.offset[i];
    p.off_out = static_cast<int32_t>(off_out);
    p.fan = fan;
    p.is_split = split_flag ? 1 : 0;
    p.shared_noise = (split_flag && !t->independent && t->coef[i].g > 0.0f) ? 1 : 0;
    p.write_children = 1;
    p.logp_out = t->buf.logp;
    cudaError_t e = launch_step(p, as_stream(stream));
    if (e != cudaSuccess) return cuda_fail(e, "step kernel");
    // this launch summed the previous level's log-probs in its prologue; its own are pending until the next
    // launch, or until the flush below when the tree is complete
    t->pending = FinalizeDesc{t->buf.logp, static_cast<int32_t>(W_out), static_cast<int32_t>(off_out), p.g, p.inv_2g2, p.logp_const};
    if (i + 1 == t->desc.T) {
        e = flush_pending(t, as_stream(stream));
        if (e != cudaSuccess) return cuda_fail(e, "log-prob flush kernel");
    }
    t->lv.fanout[i] = fan;
    t->lv.width[i + 1] = static_cast<int32_t>(W_out);
    t->lv.offset[i + 2] = static_cast<int32_t>(off_out + W_out);
    t->depth = i + 1;
    return BGRPO_OK;
}

bgrpo_status bgrpo_tree_rollout(bgrpo_tree* t, const uint8_t* split_flags_host, const void* packed_dev, int32_t hidden,
                                float* v_dev, void* stream) {
    if (!t || !split_flags_host) return fail(BGRPO_ERR_INVALID_ARG, "tree or split_flags is NULL");
    if (packed_dev && !v_dev) return fail(BGRPO_ERR_INVALID_ARG, "the MLP velocity needs a velocity buffer");
    if (!packed_dev && !t->mu) return fail(BGRPO_ERR_STATE, "no velocity: pass the packed MLP weights or bind a linear velocity");
    for (int i = t->depth; i < t->desc.T; ++i) {
        if (packed_dev) {
            const bgrpo_status st = bgrpo_velocity_mlp(t, packed_dev, hidden, v_dev, stream);
            if (st != BGRPO_OK) return st;
        }
        const bgrpo_status st = bgrpo_tree_step(t, split_flags_host[i] ? 1 : 0, packed_dev ? v_dev : nullptr, stream);
        if (st != BGRPO_OK) return st;
    }
    return BGRPO_OK;
}

bgrpo_status bgrpo_tree_rollout_fused(bgrpo_tree* t, const uint8_t* split_flags_host, void* stream) {
    if (!t || !split_flags_host) return fail(BGRPO_ERR_INVALID_ARG, "tree or split_flags is NULL");
    if (t->depth != 0) return fail(BGRPO_ERR_STATE, "the whole-tree rollout starts from a freshly initialised or reset tree");
    if (!t->mu) return fail(BGRPO_ERR_STATE, "the whole-tree rollout needs the bound closed-form velocity");
    const int T = t->desc.T;
    FusedLaunch p;
    std::memset(&p, 0, sizeof(p));
    int n_splits = 0;
    int64_t width = 1, off = 1;
    p.off[0] = 0;
    p.off[1] = 1;
    for (int i = 0; i < T; ++i) {
        const bool split = split_flags_host[i] != 0;
        if (split) {
            if (((t->ode_bits >> i) & 1ull) && t->desc.sigma > 0.0f)
                return fail(BGRPO_ERR_INVALID_ARG, "a split step must be an SDE step of the hybrid schedule");
            ++n_splits;
            p.split_bits |= 1ull << i;
            width *= t->desc.K;
        }
        off += width;
        if (off > t->desc.nodes_cap) return fail(BGRPO_ERR_CAPACITY, "children exceed nodes_cap");
        p.off[i + 2] = static_cast<int32_t>(off);
        const StepCoef& k = t->coef[i];
        p.ca[i] = k.lin_a;
        p.cb[i] = k.lin_b;
        p.g[i] = k.g;
        p.inv_2g2[i] = k.inv_2g2;
        p.logp_const[i] = k.logp_const;
    }
    if (n_splits > kFusedMaxSplits) return fail(BGRPO_ERR_UNSUPPORTED, "more split steps than the whole-tree kernel walks; use tree_step");
    p.latents = t->buf.latents;
    p.mu = t->mu;
    p.logp = t->buf.logp;
    p.table = t->buf.node_table;
    p.partialsf = t->partialsf;
    p.status = t->status;
    p.per_row_cap = static_cast<int32_t>(partials_per_row(t->D));
    p.D = t->D;
    p.n_trees = t->desc.n_trees;
    p.nodes_cap = t->desc.nodes_cap;
    p.nchunks = static_cast<int32_t>((t->D / 4 + kFusedChunkVec - 1) / kFusedChunkVec);
    p.per_row = static_cast<int32_t>(fused_partials_per_row(t->D));
    p.T = T;
    p.K = t->desc.K;
    p.shared_noise = t->independent ? 0 : 1;
    p.node_id_base = static_cast<uint32_t>(t->desc.tree_id_base * t->desc.nodes_cap);
    p.keys = make_philox_keys(t->desc.seed);
    p.mix_shared = t->mix_shared;
    p.mix_innov = t->mix_innov;
    const cudaError_t e = launch_rollout_fused(p, static_cast<int32_t>(off), as_stream(stream));
    if (e != cudaSuccess) return cuda_fail(e, "whole-tree rollout kernel");
    // host mirror of the finished tree
    int32_t w = 1;
    for (int i = 0; i < T; ++i) {
        const int fan = ((p.split_bits >> i) & 1ull) ? t->desc.K : 1;
        t->lv.fanout[i] = fan;
        w *= fan;
        t->lv.width[i + 1] = w;
        t->lv.offset[i + 2] = p.off[i + 2];
    }
    t->pending.logp_out = nullptr;
    t->depth = T;
    return BGRPO_OK;
}

bgrpo_status bgrpo_tree_logprob(bgrpo_tree* t, int32_t step, const float* v_dev, float* logp_out_dev, void* stream) {
    if (!t || !logp_out_dev) return fail(BGRPO_ERR_INVALID_ARG, "tree or output is NULL");
    if (step < -1 || step >= t->depth) return fail(BGRPO_ERR_STATE, "step has not been taken");
    if (step == -1 && v_dev) return fail(BGRPO_ERR_INVALID_ARG, "step -1 works with the bound linear velocity only");
    if (!v_dev && !t->mu) return fail(BGRPO_ERR_STATE, "no velocity: pass v_dev or bind a linear velocity");
    if (v_dev && !aligned(v_dev, 16)) return fail(BGRPO_ERR_INVALID_ARG, "v misaligned");
    const int first = step < 0 ? 0 : step, last = step < 0 ? t->depth - 1 : step;
    {   // a step's own sums may still be pending and could live in the rows this call is about to rewrite
        const cudaError_t e0 = flush_pending(t, as_stream(stream));
        if (e0 != cudaSuccess) return cuda_fail(e0, "log-prob flush kernel");
    }
    for (int i = first; i <= last; ++i) {
        StepLaunch p;
        fill_step_launch(t, i, v_dev, &p);
        p.W_in = t->lv.width[i];
        p.off_in = t->lv.offset[i];
        p.off_out = t->lv.offset[i + 1];
        p.fan = t->lv.fanout[i];
        p.is_split = 0;
        p.shared_noise = 0;
        p.write_children = 0;
        p.logp_out = logp_out_dev;
        cudaError_t e = launch_step(p, as_stream(stream));
        if (e != cudaSuccess) return cuda_fail(e, "logprob kernel");
        t->pending = FinalizeDesc{logp_out_dev, t->lv.width[i + 1], t->lv.offset[i + 1], p.g, p.inv_2g2, p.logp_const};
    }
    const cudaError_t e = flush_pending(t, as_stream(stream));
    if (e != cudaSuccess) return cuda_fail(e, "log-prob flush kernel");
    return BGRPO_OK;
}

static bgrpo_status reward_common(bgrpo_tree* t, const float* target, float scale, float* r, int mode, void* stream) {
    if (!t || !target || !r) return fail(BGRPO_ERR_INVALID_ARG, "tree, target or output is NULL");
    if (!tree_complete(t)) return fail(BGRPO_ERR_STATE, "tree is not complete");
    if (!aligned(target, 16)) return fail(BGRPO_ERR_INVALID_ARG, "target misaligned");
    RewardLaunch p;
    p.latents = t->buf.latents;
    p.target = target;
    p.r = r;
    p.partials = t->partials;
    p.counters = t->counters;
    p.status = t->status;
    p.nchunks_cap = t->nchunks;
    p.D = t->D;
    p.n_trees = t->desc.n_trees;
    p.nodes_cap = t->desc.nodes_cap;
    p.nchunks = t->nchunks_reward;
    p.leaves = t->lv.width[t->desc.T];
    p.off_leaf = t->lv.offset[t->desc.T];
    p.scale = scale;
    p.mode = mode;
    cudaError_t e = launch_reward(p, as_stream(stream));
    if (e != cudaSuccess) return cuda_fail(e, "reward kernel");
    return BGRPO_OK;
}

bgrpo_status bgrpo_leaf_reward_mse(bgrpo_tree* t, const float* target_dev, float* r_out_dev, void* stream) {
    return reward_common(t, target_dev, 0.0f, r_out_dev, 0, stream);
}
bgrpo_status bgrpo_leaf_reward_cos(bgrpo_tree* t, const float* target_dev, float scale, float* r_inout_dev, void* stream) {
    return reward_common(t, target_dev, scale, r_inout_dev, 1, stream);
}

bgrpo_status bgrpo_tree_fuse_advantage(bgrpo_tree* t, const float* leaf_rewards_dev, float beta, float logp_scale,
                                       float eps, float adv_clip_max, void* stream) {
    if (!t || !leaf_rewards_dev) return fail(BGRPO_ERR_INVALID_ARG, "tree or rewards is NULL");
    if (!tree_complete(t)) return fail(BGRPO_ERR_STATE, "tree is not complete");
    if (!std::isfinite(beta) || !std::isfinite(logp_scale) || !(eps >= 0.0f) || std::isnan(adv_clip_max))
        return fail(BGRPO_ERR_INVALID_ARG, "beta, logp_scale must be finite and eps >= 0");
    FuseLaunch p;
    p.leaf_r = leaf_rewards_dev;
    p.logp = t->buf.logp;
    p.rbar = t->buf.rbar;
    p.adv = t->buf.adv;
    p.status = t->status;
    p.node_scratch = t->node_scratch;
    p.lv = t->lv;
    p.n_trees = t->desc.n_trees;
    p.nodes_cap = t->desc.nodes_cap;
    p.T = t->desc.T;
    p.nodes = t->lv.offset[t->desc.T + 1];
    p.beta_scaled = static_cast<double>(beta) * static_cast<double>(logp_scale);
    p.eps = eps;
    p.clip = adv_clip_max;
    cudaError_t e = launch_fuse_advantage(p, as_stream(stream));
    if (e != cudaSuccess) return cuda_fail(e, "fuse kernel");
    return BGRPO_OK;
}

bgrpo_status bgrpo_tree_fusion_ess(bgrpo_tree* t, float beta, float logp_scale, float* ess_out_dev, void* stream) {
    if (!t || !ess_out_dev) return fail(BGRPO_ERR_INVALID_ARG, "tree or output is NULL");
    if (!tree_complete(t)) return fail(BGRPO_ERR_STATE, "tree is not complete");
    if (!std::isfinite(beta) || !std::isfinite(logp_scale)) return fail(BGRPO_ERR_INVALID_ARG, "beta and logp_scale must be finite");
    EssLaunch p;
    p.logp = t->buf.logp;
    p.ess = ess_out_dev;
    p.node_scratch = t->node_scratch;
    p.status = t->status;
    p.lv = t->lv;
    p.n_trees = t->desc.n_trees;
    p.nodes_cap = t->desc.nodes_cap;
    p.T = t->desc.T;
    p.nodes = t->lv.offset[t->desc.T + 1];
    p.beta_scaled = static_cast<double>(beta) * static_cast<double>(logp_scale);
    const cudaError_t e = launch_fusion_ess(p, as_stream(stream));
    if (e != cudaSuccess) return cuda_fail(e, "fusion ESS kernel");
    return BGRPO_OK;
}

bgrpo_status bgrpo_tree_prune(bgrpo_tree* t, int32_t width_mode, int32_t k_or_b, const int32_t* pruned_steps_host,
                              int32_t n_pruned, int32_t ignore_last_step, void* stream) {
    if (!t) return fail(BGRPO_ERR_INVALID_ARG, "tree is NULL");
    if (!tree_complete(t)) return fail(BGRPO_ERR_STATE, "tree is not complete");
    if (width_mode < BGRPO_WIDTH_NONE || width_mode > BGRPO_WIDTH_EXTREME_B) return fail(BGRPO_ERR_INVALID_ARG, "unknown width mode");
    if (width_mode != BGRPO_WIDTH_NONE && k_or_b < 1) return fail(BGRPO_ERR_INVALID_ARG, "k_or_b must be >= 1");
    if (n_pruned < 0 || (n_pruned > 0 && !pruned_steps_host)) return fail(BGRPO_ERR_INVALID_ARG, "bad pruned_steps");
    PruneLaunch p;
    p.pruned_bits = t->ode_bits;      // deterministic steps have no transition density: never in the edge set
    for (int q = 0; q < n_pruned; ++q) {
        if (pruned_steps_host[q] < 0 || pruned_steps_host[q] >= t->desc.T) return fail(BGRPO_ERR_INVALID_ARG, "pruned step out of range");
        p.pruned_bits |= 1ull << pruned_steps_host[q];
    }
    p.rbar = t->buf.rbar;
    p.table = t->buf.node_table;
    p.mask = t->buf.mask;
    p.status = t->status;
    p.lv = t->lv;
    p.n_trees = t->desc.n_trees;
    p.nodes_cap = t->desc.nodes_cap;
    p.T = t->desc.T;
    p.nodes = t->lv.offset[t->desc.T + 1];
    p.mode = width_mode;
    p.k = k_or_b;
    p.last_split = -1;
    for (int i = 0; i < t->desc.T; ++i)
        if (t->lv.fanout[i] > 1) p.last_split = i;
    p.ignore_last = ignore_last_step ? 1 : 0;
    cudaError_t e = launch_prune(p, as_stream(stream));
    if (e != cudaSuccess) return cuda_fail(e, "prune kernel");
    return BGRPO_OK;
}

bgrpo_status bgrpo_tree_grpo_objective(bgrpo_tree* t, const float* logp_new_dev, const float* logp_old_dev, float logp_scale,
                                       float clip_eps, float* terms_out_dev, float* J_out_dev, void* stream) {
    if (!t || !logp_new_dev || !J_out_dev) return fail(BGRPO_ERR_INVALID_ARG, "tree, logp_new or J_out is NULL");
    if (!tree_complete(t)) return fail(BGRPO_ERR_STATE, "tree is not complete");
    if (!std::isfinite(logp_scale) || !(clip_eps >= 0.0f) || !std::isfinite(clip_eps)) return fail(BGRPO_ERR_INVALID_ARG, "logp_scale must be finite and clip_eps >= 0");
    ObjectiveLaunch p;
    p.logp_new = logp_new_dev;
    p.logp_old = logp_old_dev ? logp_old_dev : t->buf.logp;
    p.adv = t->buf.adv;
    p.mask = t->buf.mask;
    p.terms = terms_out_dev;
    p.J = J_out_dev;
    p.status = t->status;
    p.n_trees = t->desc.n_trees;
    p.nodes_cap = t->desc.nodes_cap;
    p.nodes = t->lv.offset[t->desc.T + 1];
    p.logp_scale = static_cast<double>(logp_scale);
    p.clip_eps = clip_eps;
    cudaError_t e = launch_objective(p, as_stream(stream));
    return e == cudaSuccess ? BGRPO_OK : cuda_fail(e, "objective kernel");
}

bgrpo_status bgrpo_tree_set_sde_steps(bgrpo_tree* t, const uint8_t* sde_flags_host) {
    if (!t) return fail(BGRPO_ERR_INVALID_ARG, "tree is NULL");
    uint64_t ode = 0;
    if (sde_flags_host)
        for (int i = 0; i < t->desc.T; ++i)
            if (!sde_flags_host[i]) ode |= 1ull << i;
    t->ode_bits = ode;
    fill_coefficients(t);
    return BGRPO_OK;
}

bgrpo_status bgrpo_mix_sde_steps(int32_t T, const int32_t* split_steps, int32_t n_splits, int32_t iter, int32_t window,
                                 int32_t every, int32_t start, uint8_t* flags_out) {
    if (T < 1 || T > BGRPO_MAX_T || !flags_out || n_splits < 0 || (n_splits > 0 && !split_steps) || iter < 0 || window < 0 || every < 1 || start < 0)
        return fail(BGRPO_ERR_INVALID_ARG, "bad schedule arguments");
    for (int i = 0; i < T; ++i) flags_out[i] = 0;
    for (int q = 0; q < n_splits; ++q) {
        if (split_steps[q] < 0 || split_steps[q] >= T) return fail(BGRPO_ERR_INVALID_ARG, "split step out of range");
        flags_out[split_steps[q]] = 1;
    }
    int first = start + iter / every;
    const int last_first = T - window > 0 ? T - window : 0;
    if (first > last_first) first = last_first;
    for (int j = 0; j < window && first + j < T; ++j) flags_out[first + j] = 1;
    return BGRPO_OK;
}

bgrpo_status bgrpo_depth_window(int32_t iter, int32_t start, int32_t size, int32_t every, int32_t stop, int32_t* steps_out, int32_t* n_out) {
    if (!steps_out || !n_out || iter < 0 || start < 0 || size < 1 || every < 1) return fail(BGRPO_ERR_INVALID_ARG, "bad window arguments");
    if (stop >= 0 && stop - size < 0) return fail(BGRPO_ERR_INVALID_ARG, "stop leaves no room for the window");
    int first = start + iter / every;
    if (stop >= 0 && first > stop - size) first = stop - size;
    for (int j = 0; j < size; ++j) steps_out[j] = first + j;
    *n_out = size;
    return BGRPO_OK;
}

bgrpo_status bgrpo_tree_stats(const bgrpo_tree* t, int32_t* depth, int64_t* nodes, int64_t* node_steps, int64_t* model_evals, int64_t* frontier_width) {
    if (!t) return fail(BGRPO_ERR_INVALID_ARG, "tree is NULL");
    const int64_t n = t->lv.offset[t->depth + 1];
    if (depth) *depth = t->depth;
    if (nodes) *nodes = n;
    if (node_steps) *node_steps = n - 1;
    if (model_evals) *model_evals = t->lv.offset[t->depth];      // every node above the frontier was evaluated once
    if (frontier_width) *frontier_width = t->lv.width[t->depth];
    return BGRPO_OK;
}

bgrpo_status bgrpo_tree_levels(const bgrpo_tree* t, int32_t n, int32_t* widths_out, int32_t* offsets_out) {
    if (!t || n < 0 || !widths_out || !offsets_out) return fail(BGRPO_ERR_INVALID_ARG, "bad arguments");
    for (int d = 0; d <= t->depth && d < n; ++d) {
        widths_out[d] = t->lv.width[d];
        offsets_out[d] = t->lv.offset[d];
    }
    return BGRPO_OK;
}

bgrpo_status bgrpo_tree_sync_status(bgrpo_tree* t, void* stream) {
    if (!t) return fail(BGRPO_ERR_INVALID_ARG, "tree is NULL");
    int32_t word = 0;
    cudaError_t e = cudaMemcpyAsync(&word, t->status, sizeof(word), cudaMemcpyDeviceToHost, as_stream(stream));
    if (e == cudaSuccess) e = cudaMemsetAsync(t->status, 0, sizeof(word), as_stream(stream));
    if (e == cudaSuccess) e = cudaStreamSynchronize(as_stream(stream));
    if (e != cudaSuccess) return cuda_fail(e, "status read");
    if (word & kStatusOutOfBounds) return fail(BGRPO_ERR_CAPACITY, "a device-side index check failed and the access was skipped (debug build)");
    if (word & kStatusWaitTimeout) return fail(BGRPO_ERR_CUDA, "a bounded wait inside the MLP velocity kernel ran out");
    return (word & kStatusNonFinite) ? fail(BGRPO_ERR_NONFINITE, "non-finite leaf reward") : BGRPO_OK;
}

bgrpo_status bgrpo_philox_words_fill(uint64_t seed, uint32_t node_id, uint32_t step, uint32_t tag, uint32_t* out_dev, int64_t n_blocks, void* stream) {
    if (!out_dev || n_blocks < 0 || !aligned(out_dev, 16)) return fail(BGRPO_ERR_INVALID_ARG, "bad output");
    cudaError_t e = launch_philox_words(seed, node_id, step, tag, out_dev, n_blocks, as_stream(stream));
    return e == cudaSuccess ? BGRPO_OK : cuda_fail(e, "philox words kernel");
}
bgrpo_status bgrpo_philox_normal_fill(uint64_t seed, uint32_t node_id, uint32_t step, uint32_t tag, float* out_dev, int64_t n, void* stream) {
    if (!out_dev || n < 0 || n % 4 != 0 || !aligned(out_dev, 16)) return fail(BGRPO_ERR_INVALID_ARG, "bad output or n % 4 != 0");
    cudaError_t e = launch_philox_normals(seed, node_id, step, tag, out_dev, n, as_stream(stream));
    return e == cudaSuccess ? BGRPO_OK : cuda_fail(e, "philox normals kernel");
}

size_t bgrpo_velocity_mlp_packed_bytes(int32_t hidden) {
    if (hidden < BGRPO_MLP_HIDDEN_MULTIPLE || hidden % BGRPO_MLP_HIDDEN_MULTIPLE != 0) return 0;
    return mlp_packed_bytes(hidden);
}

bgrpo_status bgrpo_velocity_mlp_pack(const uint16_t* W1, const uint16_t* W2, int32_t hidden, void* packed_dev, void* stream) {
    if (!W1 || !W2 || !packed_dev) return fail(BGRPO_ERR_INVALID_ARG, "NULL pointer");
    if (hidden < BGRPO_MLP_HIDDEN_MULTIPLE || hidden % BGRPO_MLP_HIDDEN_MULTIPLE != 0) return fail(BGRPO_ERR_INVALID_ARG, "hidden must be a positive multiple of 128");
    if (!aligned(packed_dev, 1024)) return fail(BGRPO_ERR_INVALID_ARG, "packed buffer must be 1024-byte aligned");
    cudaError_t e = launch_mlp_pack(W1, W2, hidden, packed_dev, as_stream(stream));
    return e == cudaSuccess ? BGRPO_OK : cuda_fail(e, "mlp pack kernel");
}

bgrpo_status bgrpo_velocity_mlp(bgrpo_tree* t, const void* packed_dev, int32_t hidden, float* v_out_dev, void* stream) {
    if (!t || !packed_dev || !v_out_dev) return fail(BGRPO_ERR_INVALID_ARG, "NULL pointer");
    if (t->desc.channels != BGRPO_MLP_CHANNELS) return fail(BGRPO_ERR_UNSUPPORTED, "the MLP stage needs 64 channels");
    if (hidden < BGRPO_MLP_HIDDEN_MULTIPLE || hidden % BGRPO_MLP_HIDDEN_MULTIPLE != 0) return fail(BGRPO_ERR_INVALID_ARG, "hidden must be a positive multiple of 128");
    if (!aligned(packed_dev, 1024) || !aligned(v_out_dev, 16)) return fail(BGRPO_ERR_INVALID_ARG, "misaligned buffer");
    if (t->depth >= t->desc.T) return fail(BGRPO_ERR_STATE, "tree already at depth T");
    const int i = t->depth;
    cudaError_t e = launch_mlp(t->buf.latents, static_cast<int64_t>(t->desc.n_trees) * t->desc.nodes_cap * t->D, static_cast<int64_t>(t->desc.nodes_cap) * t->D, static_cast<int64_t>(t->lv.offset[i]) * t->D,
                               t->desc.n_trees, static_cast<int64_t>(t->lv.width[i]) * t->desc.tokens, packed_dev, hidden,
                               v_out_dev, t->mlp_partials, t->mlp_tickets, t->status, as_stream(stream));
    return e == cudaSuccess ? BGRPO_OK : cuda_fail(e, "mlp kernel");
}

namespace {
// Host state of a tree as it is saved: everything bgrpo_tree_import needs besides the device buffers themselves.
struct TreeBlob {
    uint32_t magic, version;
    bgrpo_tree_desc desc;                // t_grid pointer not meaningful outside the process: the values follow
    float t_grid[BGRPO_MAX_T + 1];
    LevelInfo lv;
    uint64_t ode_bits;
    int32_t depth;
    float s0;                            // 0: no linear velocity was bound
};
constexpr uint32_t kBlobMagic = 0x42475250u, kBlobVersion = 1u;      // "BGRP"
}  // namespace

size_t bgrpo_tree_export_bytes(void) { return sizeof(TreeBlob); }

bgrpo_status bgrpo_tree_export(bgrpo_tree* t, void* blob_host, size_t blob_bytes, void* stream) {
    if (!t || !blob_host) return fail(BGRPO_ERR_INVALID_ARG, "tree or blob is NULL");
    if (blob_bytes < sizeof(TreeBlob)) return fail(BGRPO_ERR_CAPACITY, "blob smaller than bgrpo_tree_export_bytes()");
    const cudaError_t e = flush_pending(t, as_stream(stream));     // the last level's log-probs become final in buffers.logp
    if (e != cudaSuccess) return cuda_fail(e, "log-prob flush kernel");
    TreeBlob b;
    std::memset(&b, 0, sizeof(b));
    b.magic = kBlobMagic;
    b.version = kBlobVersion;
    b.desc = t->desc;
    b.desc.t_grid = nullptr;
    std::memcpy(b.t_grid, t->t_grid, sizeof(b.t_grid));
    b.lv = t->lv;
    b.ode_bits = t->ode_bits;
    b.depth = t->depth;
    b.s0 = t->mu ? t->s0 : 0.0f;
    std::memcpy(blob_host, &b, sizeof(b));
    return BGRPO_OK;
}

bgrpo_status bgrpo_tree_import(const void* blob_host, size_t blob_bytes, const bgrpo_buffers* buffers, void* stream, bgrpo_tree** out) {
    if (!blob_host || !buffers || !out) return fail(BGRPO_ERR_INVALID_ARG, "blob, buffers or out is NULL");
    if (blob_bytes < sizeof(TreeBlob)) return fail(BGRPO_ERR_INVALID_ARG, "blob too small");
    TreeBlob b;
    std::memcpy(&b, blob_host, sizeof(b));
    if (b.magic != kBlobMagic || b.version != kBlobVersion) return fail(BGRPO_ERR_INVALID_ARG, "not a tree blob of this library version");
    b.desc.t_grid = b.t_grid;
    bgrpo_status st = check_desc(&b.desc);
    if (st != BGRPO_OK) return st;
    if (b.depth < 0 || b.depth > b.desc.T || b.lv.offset[b.depth + 1] > b.desc.nodes_cap) return fail(BGRPO_ERR_INVALID_ARG, "blob describes a tree that does not fit its own description");
    if (!buffers->latents || !buffers->node_table || !buffers->logp || !buffers->rbar || !buffers->adv || !buffers->mask || !buffers->scratch)
        return fail(BGRPO_ERR_INVALID_ARG, "a device buffer is NULL");
    if (!aligned(buffers->latents, 16) || !aligned(buffers->scratch, 256)) return fail(BGRPO_ERR_INVALID_ARG, "misaligned device buffer");
    if (buffers->scratch_bytes < scratch_bytes_of(&b.desc)) return fail(BGRPO_ERR_CAPACITY, "scratch_bytes too small");
    bgrpo_tree* t = new (std::nothrow) bgrpo_tree();
    if (!t) return fail(BGRPO_ERR_INVALID_ARG, "out of host memory");
    t->desc = b.desc;
    std::memcpy(t->t_grid, b.t_grid, sizeof(t->t_grid));
    t->desc.t_grid = t->t_grid;
    bind_buffers(t, buffers);
    t->lv = b.lv;
    t->ode_bits = b.ode_bits;
    t->depth = b.depth;
    fill_coefficients(t);
    // the status word and the MLP tile tickets live in scratch, which may be a fresh allocation: both start at zero
    cudaError_t e = cudaMemsetAsync(t->status, 0, sizeof(int32_t), as_stream(stream));
    if (e == cudaSuccess && t->mlp_tickets) e = cudaMemsetAsync(t->mlp_tickets, 0, kMlpTicketBytes, as_stream(stream));
    if (e != cudaSuccess) {
        delete t;
        return cuda_fail(e, "clearing the status word and the MLP tickets");
    }
    *out = t;
    return BGRPO_OK;
}

bgrpo_status bgrpo_debug_bounds(bgrpo_tree* t, int32_t trip, void* stream) {
#ifdef BGRPO_DEBUG_BOUNDS
    if (trip) {
        if (!t) return fail(BGRPO_ERR_INVALID_ARG, "tree is NULL");
        const cudaError_t e = launch_debug_trip(t->status, as_stream(stream));
        if (e != cudaSuccess) return cuda_fail(e, "debug trip kernel");
    }
    return BGRPO_OK;
#else
    (void)t; (void)trip; (void)stream;
    return fail(BGRPO_ERR_UNSUPPORTED, "this library was built without device-side index checks");
#endif
}

void bgrpo_tree_destroy(bgrpo_tree* t) { delete t; }

}  // extern "C"
