/*
 * bgrpo.h - C ABI of the BranchGRPO tree-rollout / tree-reduction library (sm_100a).
 *
 * One prompt grows one rollout tree: a root noise, T reverse-SDE denoising steps, and at
 * scheduled split steps every live state forks into K children that share the prefix
 * (Branch Rollout Algorithm; Eq. 2; Algorithm 1 "Build rollout tree").  Leaf rewards are
 * fused upward into node values (Eq. 3), standardised per depth into edge advantages
 * (Eq. 4), and width/depth pruning selects the node-steps that receive gradients
 * ("Pruning Strategies").  This header declares exactly those operations.
 *
 * Conventions
 *  - Every function returns a bgrpo_status and never throws.  Nothing here allocates or
 *    frees device memory and, unless its name ends in _sync, nothing waits for the stream:
 *    work is enqueued on the `stream` argument (a cudaStream_t passed as void*; NULL is the
 *    default stream).
 *  - "device" pointers are CUDA global-memory addresses of the current device, "host"
 *    pointers are ordinary process memory.  Device buffers are owned by the caller and
 *    must outlive the handle; they must be 16-byte aligned.
 *  - Step index i counts from the noise end: t_grid[0] is the noisiest time, step i is the
 *    transition t_i -> t_{i+1}, node depth d is the number of steps taken.
 *  - Nodes of one tree are stored in level order.  If depth d starts at local index off_d
 *    and holds W_d nodes, the children of its j-th node are the nodes j*F + b of depth d+1
 *    (F = K at a split step, 1 otherwise).  Tree t owns rows [t*nodes_cap, (t+1)*nodes_cap)
 *    of every per-node buffer.
 *  - Noise is counter based (Philox4x32-10, Salmon et al. SC'11): key = the 64-bit seed,
 *    counter = (element/4, global node id, step, stream tag) with global node id =
 *    (tree_id_base + t) * nodes_cap + local index.  Tag 0: root latent (root id, step 0);
 *    tag 1: the shared xi_0 of Eq. 2 (parent id); tag 2: the innovation eta_b of Eq. 2 and
 *    the noise of every non-split step (child id).  A 32-bit word x maps to the uniform
 *    ((x >> 9) + 0.5) * 2^-23; word pairs (0,1) and (2,3) of a block give the normals
 *    r cos(2 pi u_b), r sin(2 pi u_b), r = sqrt(-2 ln u_a), for elements 4*(e/4)+0..3.
 */
#ifndef BGRPO_H_
#define BGRPO_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define BGRPO_MAX_T 64      /* most denoising steps per tree */
#define BGRPO_MAX_K 4       /* largest branching factor */
#define BGRPO_MLP_CHANNELS 64
#define BGRPO_MLP_HIDDEN_MULTIPLE 128

typedef enum {
    BGRPO_OK = 0,
    BGRPO_ERR_INVALID_ARG = 1,   /* NULL pointer, size or value out of range, misaligned buffer */
    BGRPO_ERR_STATE = 2,         /* call out of order: step past depth T, reductions before the tree is complete */
    BGRPO_ERR_CAPACITY = 3,      /* nodes_cap, scratch_bytes or a node-id range too small for this tree */
    BGRPO_ERR_NONFINITE = 4,     /* a kernel met a NaN/Inf leaf reward (reported by bgrpo_tree_sync_status) */
    BGRPO_ERR_CUDA = 5,          /* a CUDA runtime call or launch failed */
    BGRPO_ERR_UNSUPPORTED = 6    /* valid request outside what the kernels cover */
} bgrpo_status;

/* Width-pruning modes ("Width Pruning"; ablation "Pruning Strategies"). */
enum {
    BGRPO_WIDTH_NONE = 0,
    BGRPO_WIDTH_PER_SPLIT_TOPK = 1,   /* keep the k best children of every parent at every split */
    BGRPO_WIDTH_LAST_SPLIT_TOPK = 2,  /* Parent-Top1 (k = 1): only at the last branching step */
    BGRPO_WIDTH_EXTREME_B = 3         /* keep the b best and the b worst leaves (root paths) */
};

/* Philox stream tags. */
enum { BGRPO_TAG_ROOT = 0, BGRPO_TAG_SHARED = 1, BGRPO_TAG_INNOV = 2 };

typedef struct bgrpo_tree bgrpo_tree;    /* opaque host-side handle */

/* Problem description ("Preliminaries": depth T, branching factor K, branch correlation s). */
typedef struct {
    int32_t  n_trees;        /* prompts in this batch (>= 1) */
    int32_t  tokens;         /* latent elements per node D = tokens * channels, D % 4 == 0 */
    int32_t  channels;
    int32_t  T;              /* denoising steps = tree depth, 1..BGRPO_MAX_T */
    int32_t  K;              /* children per split, 1..BGRPO_MAX_K */
    int32_t  nodes_cap;      /* rows reserved per tree in every per-node buffer (>= nodes of the tree) */
    int64_t  tree_id_base;   /* global index of this batch's first tree (shards of one job draw the same noise) */
    float    sigma;          /* diffusion g(t) = sigma ("Eta"); 0 = deterministic steps, log-probs written as 0 */
    float    branch_corr_s;  /* s of Eq. 2; +INF (or < 0) = independent children xi_b = eta_b */
    uint64_t seed;           /* Philox key */
    const float* t_grid;     /* host, T+1 values, strictly decreasing, t_grid[0] <= 1, t_grid[T-1] > 0, t_grid[T] >= 0 */
} bgrpo_tree_desc;

/* Device buffers of one batch of trees, all caller-owned. */
typedef struct {
    float*   latents;     /* device [n_trees][nodes_cap][D] float32 latent pool */
    int32_t* node_table;  /* device [4][n_trees*nodes_cap]: parent (local, -1 root) | depth | split_step (-1 none) | branch_id */
    float*   logp;        /* device [n_trees][nodes_cap]: log-prob of the edge INTO each node (root: 0) */
    float*   rbar;        /* device [n_trees][nodes_cap]: fused value (Eq. 3) */
    float*   adv;         /* device [n_trees][nodes_cap]: advantage of the edge into each node (Eq. 4; root: 0) */
    uint8_t* mask;        /* device [n_trees][nodes_cap]: 1 = the node-step receives gradients */
    void*    scratch;     /* device, >= scratch_bytes of bgrpo_tree_workspace, 256-byte aligned; kernels keep reduction partials, counters and a status word here */
    size_t   scratch_bytes;
} bgrpo_buffers;

typedef struct {
    size_t latents_bytes;         /* n_trees * nodes_cap * D * 4 */
    size_t node_table_bytes;      /* 4 * n_trees * nodes_cap * 4 */
    size_t per_node_float_bytes;  /* n_trees * nodes_cap * 4: each of logp, rbar, adv */
    size_t mask_bytes;            /* n_trees * nodes_cap */
    size_t scratch_bytes;
} bgrpo_sizes;

/* Sizes of the buffers a description needs.  Host only.  INVALID_ARG on a bad description. */
bgrpo_status bgrpo_tree_workspace(const bgrpo_tree_desc* desc, bgrpo_sizes* out);

/* Node bookkeeping of a schedule (Table 1 caption: per-sample NFE = evaluations of the tree / final samples).
 * split_steps: host array of n_splits distinct steps in 0..T-1.  Any output may be NULL.
 * nodes = sum_d W_d; node_steps = nodes - 1 (edges); model_evals = nodes - leaves (one velocity per parent). */
bgrpo_status bgrpo_tree_count(int32_t T, int32_t K, const int32_t* split_steps, int32_t n_splits,
                              int64_t* nodes, int64_t* node_steps, int64_t* model_evals, int64_t* leaves);

/* tree_init (Algorithm 1, "Sample root noise"; "Init same noise"): validates, creates the handle, and enqueues the
 * kernel that writes each tree's root row of the node table and its root latent z_0 ~ N(0, I) (tag ROOT).
 * *out is set only on BGRPO_OK.  Errors: INVALID_ARG, CAPACITY (scratch or node-id range), CUDA. */
bgrpo_status bgrpo_tree_init(const bgrpo_tree_desc* desc, const bgrpo_buffers* buffers, void* stream, bgrpo_tree** out);

/* Restart the same handle at depth 0 with a new seed (same buffers): enqueues the root kernel again. */
bgrpo_status bgrpo_tree_reset(bgrpo_tree* tree, uint64_t seed, void* stream);

/* Closed-form velocity of the rectified-flow path towards a Gaussian target N(mu, s0^2 I):
 * v(z,t) = -mu + k_t (z - (1-t) mu), k_t = (t - (1-t) s0^2) / ((1-t)^2 s0^2 + t^2).
 * mu_dev: device [n_trees][D].  Host only; later steps with v_dev == NULL use it. */
bgrpo_status bgrpo_velocity_linear_bind(bgrpo_tree* tree, const float* mu_dev, float s0);

/* tree_step: one denoising step of every live node, depth i -> i+1 (Eq. 2; appendix, Euler-Maruyama form
 * z_{i+1} = mu_theta(z_i, t_i) + g_i xi, g_i = sigma sqrt(h_i)).  split_flag != 0 forks each node into K children with
 * xi_b = (xi_0 + s eta_b)/sqrt(1+s^2); otherwise one child with xi = eta.  The mean is the reverse-time Euler step of
 * the rectified-flow SDE, mu_theta = z - h v - (sigma^2 h / (2 t)) (z + (1-t) v), evaluated once per parent.
 * v_dev: device [n_trees][W_i][D] velocities of the current frontier (e.g. from bgrpo_velocity_mlp), or NULL for the
 * bound linear velocity.  One fused kernel appends the children's node-table rows, writes their latents and the
 * partial sums of the per-element-mean Gaussian log-prob of each new edge,
 *   logp = -(1/D) sum_e (z'_e - mu_e)^2 / (2 g_i^2) - ln g_i - 0.5 ln(2 pi)      (multiply by D for the joint density).
 * The value is stored as float32: its rounding (about 1e-7 at |logp| ~ 1) is multiplied by whatever scale a caller
 * applies later, so logp_scale = D in tree_fuse_advantage / tree_grpo_objective gives joint densities good to about
 * 1e-7 * D in the exponent - fine for D up to a few thousand, meaningless at D ~ 1e5 (use a scale of order 1 there, as the
 * workloads do).  At step time the squared residual is taken as g^2 xi^2 from the drawn noise, tree_logprob takes it
 * from the stored child; the two agree to the rounding of the child (test: rho = 1 within 1e-5).
 * The sums are completed, in a fixed order, by the next call for this tree that is enqueued on the stream (the next
 * tree_step's kernel does it in its prologue) and at the latest by the step that completes the tree, which enqueues a
 * small flush kernel: buffers.logp of a level is final once one of those has run.  Use one stream per tree handle.
 * Errors: STATE (already at depth T; NULL v_dev without a bound velocity), CAPACITY (children exceed nodes_cap), CUDA. */
bgrpo_status bgrpo_tree_step(bgrpo_tree* tree, int32_t split_flag, const float* v_dev, void* stream);

/* tree_rollout: the remaining steps of the tree, depth .. T-1, in one host call (Algorithm 1, "Build rollout tree": for
 * every step, the velocity of every live node, then the step that forks or advances it).  The same kernels in the same
 * order as calling bgrpo_velocity_mlp (when packed_dev is given) and bgrpo_tree_step step by step, so every output is
 * identical bit for bit; what it saves is the caller's per-call overhead, which on single-tree workloads (launches of
 * 5-40 us) is comparable to the launches themselves.
 *   split_flags_host  host array of T flags (indexed by step), non-zero = fork every node into K children
 *   packed_dev        device, packed MLP weights (bgrpo_velocity_mlp_pack), or NULL for the bound linear velocity
 *   v_dev             device [n_trees][W_max][D] float32 scratch for the velocities of the widest frontier (NULL allowed
 *                     with packed_dev == NULL)
 * Errors: those of the two calls (the tree keeps the depth it reached); INVALID_ARG, STATE as stated for them. */
bgrpo_status bgrpo_tree_rollout(bgrpo_tree* tree, const uint8_t* split_flags_host, const void* packed_dev, int32_t hidden,
                                float* v_dev, void* stream);

/* tree_rollout_fused: all T steps of tree_step in one launch, for the bound closed-form velocity (Branch Rollout
 * Algorithm, where a prefix is computed once for all the leaves below it; Eq. 2; Algorithm 1 "Build rollout tree").
 * That velocity acts on every latent
 * element by itself, so one thread can carry its elements from the root to every leaf, depth first, and write each
 * node once: nothing is read back between depths.  Call it on a freshly initialised or reset tree.  split_flags_host:
 * host array of T flags, non-zero = step i forks every node into K children.  Latents, node table and log-probs are the
 * ones T calls of tree_step give (latents and table bit for bit; log-probs up to the order of a float32 partial sum),
 * and buffers.logp is final when the call's kernels have run.  At most 6 split steps.
 * Errors: STATE (tree not at depth 0, no bound linear velocity), CAPACITY (tree exceeds nodes_cap), UNSUPPORTED (more
 * than 6 split steps: use tree_step), INVALID_ARG (a split on an ODE step of the hybrid schedule), CUDA. */
bgrpo_status bgrpo_tree_rollout_fused(bgrpo_tree* tree, const uint8_t* split_flags_host, void* stream);

/* tree_logprob: log pi(z_child | z_parent) of stored edges under a GIVEN velocity (the numerator of rho_e in Eq. 5;
 * under the behaviour velocity it reproduces the step-time values, the summands of s_l in Eq. 3).
 * step >= 0: the edges of that step, v_dev = device [n_trees][W_step][D] or NULL (bound linear velocity).
 * step == -1: every edge taken so far, bound linear velocity only (v_dev must be NULL).
 * logp_out_dev: device [n_trees][nodes_cap], indexed like buffers.logp; only the addressed edges are written. */
bgrpo_status bgrpo_tree_logprob(bgrpo_tree* tree, int32_t step, const float* v_dev, float* logp_out_dev, void* stream);

/* Per-token MLP stand-in for the denoiser: v = bf16(GELU(bf16(z) W1)) W2, bf16 operands, float32 accumulation, float32
 * output, evaluated for every node of the CURRENT frontier on tcgen05 tensor cores.  channels must be 64 and hidden a
 * multiple of 128.  bgrpo_velocity_mlp_pack reorders the weights once into the tiled shared-memory image the kernel
 * streams (packed_dev: device, bgrpo_velocity_mlp_packed_bytes(hidden) bytes, 1024-byte aligned).
 * W1_bf16_dev: device [64][hidden] bf16 bits; W2_bf16_dev: device [hidden][64] bf16 bits.
 * v_out_dev: device [n_trees][W_i][D] float32.  Frontiers of fewer 128-token tiles than SMs are cut along the hidden
 * dimension as well; the partial sums of that split live in the tree's scratch (the workspace query accounts for them)
 * and are added in a fixed order, so repeated calls give identical bits. */
size_t       bgrpo_velocity_mlp_packed_bytes(int32_t hidden);
bgrpo_status bgrpo_velocity_mlp_pack(const uint16_t* W1_bf16_dev, const uint16_t* W2_bf16_dev, int32_t hidden,
                                     void* packed_dev, void* stream);
bgrpo_status bgrpo_velocity_mlp(bgrpo_tree* tree, const void* packed_dev, int32_t hidden, float* v_out_dev, void* stream);

/* Leaf-reward stand-ins (the paper's reward models are outside the library; Algorithm 1 "Evaluate rewards for leaves").
 * target_dev: device [n_trees][D].  r_*_dev: device [n_trees][leaves] float32.
 * mse: r = -mean_e (z_leaf - target)^2.   cos: r += scale * <z_leaf,target>/(|z_leaf||target|) (adds to r_inout).
 * STATE unless the tree is complete (depth T). */
bgrpo_status bgrpo_leaf_reward_mse(bgrpo_tree* tree, const float* target_dev, float* r_out_dev, void* stream);
bgrpo_status bgrpo_leaf_reward_cos(bgrpo_tree* tree, const float* target_dev, float scale, float* r_inout_dev, void* stream);

/* tree_fuse_advantage: reward fusion (Eq. 3) then depth-wise normalisation (Eq. 4), one kernel.
 * rbar(n) = sum_{l in L(n)} softmax_l(beta * logp_scale * s_l) r_l with s_l the sum of buffers.logp along n -> l
 * (beta = 0: uniform mean); A(n) = (rbar(n) - mean_d) / (std_d + eps) over the nodes of depth d of the same tree
 * (population std; a single-node depth gives 0), clipped to [-adv_clip_max, adv_clip_max] when adv_clip_max > 0.
 * leaf_rewards_dev: device [n_trees][leaves] float32.  Writes buffers.rbar and buffers.adv (root advantage 0).
 * A non-finite reward sets the NONFINITE status word and writes NaN for that tree. STATE unless the tree is complete. */
bgrpo_status bgrpo_tree_fuse_advantage(bgrpo_tree* tree, const float* leaf_rewards_dev, float beta, float logp_scale,
                                       float eps, float adv_clip_max, void* stream);

/* Effective sample size of the fusion weights of every node (appendix "Reward Fusion: Unbiasedness and Variance
 * Reduction"): ESS(n) = (sum_l w_l)^2 / sum_l w_l^2 over the descendant leaves l of n, with the weights of Eq. 3,
 * w_l = exp(beta * logp_scale * s_l).  A diagnostic of how far path-probability weighting concentrates on a few leaves:
 * beta = 0 gives the number of descendant leaves, one dominant leaf gives 1.  Reads buffers.logp of a complete tree.
 * ess_out_dev: device [n_trees][nodes_cap] float32. */
bgrpo_status bgrpo_tree_fusion_ess(bgrpo_tree* tree, float beta, float logp_scale, float* ess_out_dev, void* stream);

/* tree_prune: gradient mask per node-step; reads buffers.rbar, writes buffers.mask only (section "Pruning Strategies":
 * pruning selects what is back-propagated and leaves rollouts, rewards and advantages as they are).  mask(n) = keep_width(n) AND step(depth(n)-1) not in
 * pruned_steps AND n is not the root AND (ignore_last_step == 0 OR depth(n) < T).  Width ranking compares the float32
 * rbar values, ties to the lower branch (or leaf) index; a pruned child masks its whole subtree.
 * pruned_steps_host: host array of n_pruned steps in 0..T-1 (the set D of "Depth Pruning"), may be NULL if 0. */
bgrpo_status bgrpo_tree_prune(bgrpo_tree* tree, int32_t width_mode, int32_t k_or_b, const int32_t* pruned_steps_host,
                              int32_t n_pruned, int32_t ignore_last_step, void* stream);

/* Clipped GRPO objective over the tree's edges, forward value (Eq. 5):
 *   J = 1/|E| sum_e min(rho_e A(e), clip(rho_e, 1 - clip_eps, 1 + clip_eps) A(e)),  rho_e = exp(logp_scale (logp_new(e) - logp_old(e))),
 * per tree, with E the node-steps whose buffers.mask is 1 and A = buffers.adv (so call it after tree_fuse_advantage and
 * tree_prune).  logp_new_dev: device [n_trees][nodes_cap], e.g. from bgrpo_tree_logprob under the new policy's velocity;
 * logp_old_dev: the behaviour policy's log-probs, NULL = buffers.logp; logp_scale: D turns per-element means into joint
 * log-densities.  terms_out_dev: device [n_trees][nodes_cap] per-edge summands (0 where the mask is 0), may be NULL;
 * J_out_dev: device [n_trees] float32 (0 for a tree with no masked edge).  STATE unless the tree is complete. */
bgrpo_status bgrpo_tree_grpo_objective(bgrpo_tree* tree, const float* logp_new_dev, const float* logp_old_dev, float logp_scale,
                                       float clip_eps, float* terms_out_dev, float* J_out_dev, void* stream);

/* Hybrid ODE-SDE schedule (ablation "Hybrid ODE-SDE": split steps stay stochastic, a sliding window names further
 * stochastic steps, every other step is deterministic).  sde_flags_host: host array of T bytes, 1 = step i is
 * stochastic, 0 = deterministic (sigma = 0 for that step: drift -v only, no noise drawn, log-prob written as 0, and
 * tree_prune masks its node-steps); NULL restores "every step is SDE".  Host only; affects the steps taken afterwards.
 * A later tree_step with split_flag != 0 on an ODE step returns INVALID_ARG (identical children carry no signal). */
bgrpo_status bgrpo_tree_set_sde_steps(bgrpo_tree* tree, const uint8_t* sde_flags_host);
/* The schedule itself: flags_out[i] = 1 for every split step and for the window steps
 * min(start + iter/every, T - window) + 0..window-1.  Host only; flags_out holds T bytes. */
bgrpo_status bgrpo_mix_sde_steps(int32_t T, const int32_t* split_steps, int32_t n_splits, int32_t iter, int32_t window,
                                 int32_t every, int32_t start, uint8_t* flags_out);

/* Sliding-window schedule of depth pruning (ablation "Pruning Strategies": the window starts at the last split step,
 * spans four steps and moves one step deeper every thirty iterations, up to a stop depth): steps_out[j] = min(start + iter/every, stop-size) + j.
 * stop < 0 = no stop.  Host only; steps_out holds `size` entries. */
bgrpo_status bgrpo_depth_window(int32_t iter, int32_t start, int32_t size, int32_t every, int32_t stop,
                                int32_t* steps_out, int32_t* n_out);

/* Counters of the tree grown so far.  Any output may be NULL. */
bgrpo_status bgrpo_tree_stats(const bgrpo_tree* tree, int32_t* depth, int64_t* nodes, int64_t* node_steps,
                              int64_t* model_evals, int64_t* frontier_width);
/* Level layout: writes min(depth+1, n) widths and offsets (host arrays). */
bgrpo_status bgrpo_tree_levels(const bgrpo_tree* tree, int32_t n, int32_t* widths_out, int32_t* offsets_out);

/* Copies the device status word to the host and waits for `stream`: BGRPO_OK, BGRPO_ERR_NONFINITE (a kernel met a
 * NaN/Inf leaf reward), BGRPO_ERR_CUDA (a bounded wait inside the MLP velocity kernel ran out) or, in the debug build,
 * BGRPO_ERR_CAPACITY (a device-side index check failed; the access was skipped).  The word is cleared afterwards. */
bgrpo_status bgrpo_tree_sync_status(bgrpo_tree* tree, void* stream);

/* Saving and restoring a tree (no counterpart in the paper's method; its training loop checkpoints every 40 steps,
 * hyper-parameter table).  A tree's state is the caller's device buffers plus a small host record: description, t-grid,
 * level layout, hybrid-schedule flags, depth.  bgrpo_tree_export first enqueues the kernel that completes any pending
 * log-prob sums (so buffers.logp is final once `stream` has run), then writes the record to blob_host
 * (bgrpo_tree_export_bytes() bytes).  bgrpo_tree_import builds a new handle from such a record and a set of buffers that
 * hold what the exported tree's buffers held (the same allocations, or copies made after `stream` had run; scratch may be
 * fresh), without launching a kernel; it clears the status word and the MLP stage's tickets on `stream`.  A bound linear
 * velocity is a device pointer and is not saved: call bgrpo_velocity_linear_bind again.  Continuing an imported tree gives
 * the bits an uninterrupted tree gives.  Errors: INVALID_ARG (NULL, foreign or inconsistent record, misaligned buffer),
 * CAPACITY (blob or scratch too small), CUDA. */
size_t       bgrpo_tree_export_bytes(void);
bgrpo_status bgrpo_tree_export(bgrpo_tree* tree, void* blob_host, size_t blob_bytes, void* stream);
bgrpo_status bgrpo_tree_import(const void* blob_host, size_t blob_bytes, const bgrpo_buffers* buffers, void* stream, bgrpo_tree** out);

/* Debug build with device-side index checks (library compiled with -DBGRPO_DEBUG_BOUNDS; no counterpart in the paper).
 * In that build every kernel tests the row, chunk and element indices it derives against the extents it was launched
 * with; a failed test sets a bit of the status word and the access is skipped - nothing traps - and
 * bgrpo_tree_sync_status then returns BGRPO_ERR_CAPACITY.  bgrpo_debug_bounds returns BGRPO_OK in such a build and
 * BGRPO_ERR_UNSUPPORTED in the normal one; with trip != 0 it also enqueues a one-warp kernel that fails one such test on
 * purpose (it touches no memory), so the reporting path can be checked. */
bgrpo_status bgrpo_debug_bounds(bgrpo_tree* tree, int32_t trip, void* stream);

/* Test hooks for the noise definition above: raw Philox words (n_blocks x 4 uint32) and normals (n floats,
 * n % 4 == 0) of one (seed, node id, step, tag), starting at element 0. */
bgrpo_status bgrpo_philox_words_fill(uint64_t seed, uint32_t node_id, uint32_t step, uint32_t tag, uint32_t* out_dev,
                                     int64_t n_blocks, void* stream);
bgrpo_status bgrpo_philox_normal_fill(uint64_t seed, uint32_t node_id, uint32_t step, uint32_t tag, float* out_dev,
                                      int64_t n, void* stream);

/* bgrpo_reward_mse_static - no counterpart in the paper; a deployment convenience.
 * Some callers cannot give the library device scratch, because they cannot allocate device memory at the point where
 * they call it: a serving or training process that handed all device memory to its own pool at start-up, a plug-in
 * that runs inside another framework's step and must not trigger the device-wide synchronisation cudaMalloc implies,
 * code under a fixed memory budget.  The tree handle of bgrpo_tree_init needs a caller-allocated scratch buffer, so
 * those callers get this one self-contained call: r_out[i] = -mean_e (rows[i][e] - target[e])^2, the same reduction as
 * bgrpo_leaf_reward_mse, with the reduction partials and ticket counters kept in a fixed BGRPO_STATIC_SCRATCH_BYTES
 * array that is part of the library image (every GPU that loads the library holds that much until the process exits).
 *   rows_dev   device [n_rows][D] float32, 16-byte aligned (e.g. the leaf rows of a latent pool)
 *   target_dev device [D] float32, 16-byte aligned, shared by all rows
 *   r_out_dev  device [n_rows] float32
 * Limits: n_rows <= BGRPO_STATIC_MAX_ROWS and n_rows * ceil(D / 4096) <= (BGRPO_STATIC_SCRATCH_BYTES -
 * 4 * BGRPO_STATIC_MAX_ROWS) / 8; anything larger returns BGRPO_ERR_CAPACITY and launches nothing (split the rows
 * over several calls, one after the other).  D must be a positive multiple of 4 (INVALID_ARG otherwise).
 * The call allocates and frees nothing.  The first call on each device looks up the array's device address (a host
 * symbol lookup, done once per device with that device current); make that first call outside any stream capture.
 * All calls on a device share the one array and it keeps the previous call's contents: the call clears the counters
 * it needs on `stream` before its kernel, but two calls that can overlap on the GPU (different streams without an
 * ordering between them) race on it and give wrong results - keep calls stream-ordered. */
#define BGRPO_STATIC_SCRATCH_BYTES (512 * 1024)
#define BGRPO_STATIC_MAX_ROWS 1024
bgrpo_status bgrpo_reward_mse_static(const float* rows_dev, const float* target_dev, int32_t n_rows, int64_t D,
                                     float* r_out_dev, void* stream);

void        bgrpo_tree_destroy(bgrpo_tree* tree);
const char* bgrpo_status_string(bgrpo_status status);
/* Last CUDA error text seen by this thread's most recent failing call ("" if none). */
const char* bgrpo_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* BGRPO_H_ */
