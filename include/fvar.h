/*
 * libfvar -- late-scale step of VAR next-scale prediction under FasterVAR, for NVIDIA B200 (sm_100a).
 *
 * One call, fvar_scale_step, runs a stack of AdaLN transformer blocks over the tokens of one
 * scale; the current scale's rows attend over a multi-scale KV cache.  It runs either densely or
 * under the paper's fidelity-refinement approximation: null-prompt-only CFG (Sec. 3.2, "Semantic
 * irrelevance"), random projection of the M token rows to r rows (Sec. 3.3 "Random Projection";
 * Algorithm 1), the block forward on r rows, and representative token restoration (Sec. 3.3
 * "RTR", Eq. "upcache" and Eq. "redefine").
 *
 * Conventions
 *   - "dev" pointers are device memory of the current CUDA device, "host" pointers are host memory.
 *   - bf16 arrays are raw 16-bit patterns.  All matrices are row-major.
 *   - Weight matrices are stored [out_features][in_features] (y = x W^T + b).
 *   - The library never allocates or frees device memory and never synchronises unless a function
 *     says so; all work is enqueued on the stream given to fvar_init.  The caller owns weights,
 *     tokens, outputs, workspace and the stream, and keeps them alive while the context exists.
 *   - Every function returns an fvar_status; nothing is thrown across this boundary.  Errors found
 *     by a kernel (a bounded wait that ran out) are recorded in a device status word that
 *     fvar_poll_status reads after the caller has synchronised.
 *   - A CFG pair is two adjacent batch elements: element 2p is the prompt-conditioned branch,
 *     element 2p+1 the null-prompt branch.
 */
#ifndef FVAR_H_
#define FVAR_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct fvar_ctx fvar_ctx;

typedef enum {
  FVAR_OK = 0,
  FVAR_EINVAL = 1,       /* bad argument */
  FVAR_ENOMEM = 2,       /* workspace too small */
  FVAR_ESTATE = 3,       /* call out of order (see each function) */
  FVAR_ECUDA = 4,        /* a CUDA runtime / driver call failed */
  FVAR_ETIMEOUT = 5,     /* a bounded device-side wait ran out (fvar_poll_status) */
  FVAR_EUNSUPPORTED = 6  /* shape outside what the kernels support */
} fvar_status;

enum { FVAR_DENSE = 0, FVAR_LOWRANK_RTR = 1, FVAR_SKIP = 2 };      /* fvar_keep_policy.mode     */
enum { FVAR_CFG_PAIR = 0, FVAR_CFG_NULL_ONLY = 1 };                /* fvar_keep_policy.cfg_mode */
enum { FVAR_SELECT_TOPR = 0, FVAR_SELECT_SAMPLE = 1 };             /* fvar_keep_policy.select   */
enum { FVAR_RESTORE_RTR = 0, FVAR_RESTORE_LLS = 1 };               /* fvar_keep_policy.restore  */

/* Static shape of the block stack. */
typedef struct {
  int n_blocks;          /* transformer blocks                                                */
  int blocks_per_group;  /* RP / RTR are applied per block group (Sec. 3.3: block-level application) */
  int width;             /* C (the paper's d); multiple of 64                                 */
  int n_heads;           /* H                                                                 */
  int head_dim;          /* D: 64 or 128; H * D == C                                          */
  int ffn_dim;           /* F; multiple of 64                                                 */
  int n_scales;
  const int *scale_hw;   /* host, 2 * n_scales ints: h_k, w_k (h != w is legal)               */
  int max_batch;         /* largest B given to fvar_set_cond                                  */
  int has_cross_attn;    /* 1: blocks also cross-attend to ctx_len context tokens             */
  int ctx_len;
  int ctx_width;         /* multiple of 64                                                    */
  float ln_eps;          /* LayerNorm epsilon (1e-6 in the reference workloads)               */
} fvar_cfg;

/* Per-block parameters: each member is a host array of n_blocks device pointers to bf16 data.
 * w_qkv [3C][C], b_qkv [3C], w_o [C][C], b_o [C], w_fc1 [F][C], b_fc1 [F], w_fc2 [C][F], b_fc2 [C],
 * w_ada [6C][C], b_ada [6C] (chunks shift1, scale1, gate1, shift2, scale2, gate2);
 * cross-attention (NULL arrays when has_cross_attn == 0): w_cq [C][C], w_ckv [2C][ctx_width]
 * (keys then values), w_co [C][C], ln_c_gamma [C]. */
typedef struct {
  const void *const *w_qkv, *const *b_qkv, *const *w_o, *const *b_o;
  const void *const *w_fc1, *const *b_fc1, *const *w_fc2, *const *b_fc2;
  const void *const *w_ada, *const *b_ada;
  const void *const *w_cq, *const *w_ckv, *const *w_co, *const *ln_c_gamma;
} fvar_weights;

/* Per-call policy of a scale step. */
typedef struct {
  int mode;                   /* FVAR_DENSE | FVAR_LOWRANK_RTR | FVAR_SKIP                         */
  int cfg_mode;               /* FVAR_CFG_PAIR: all B elements; FVAR_CFG_NULL_ONLY: elements 2p+1  */
  const int *rank_per_group;  /* host, n_groups ints: r per block group; NULL -> keep_ratio        */
  float keep_ratio;           /* r = floor(keep_ratio * M + 0.5) for every group                   */
  const int *forced_indices;  /* dev, test hook: [n_groups][B_eff][r_max] ascending row indices that
                                 replace the selection (r_max = largest r of the call); NULL in production */
  int select;                 /* FVAR_SELECT_TOPR: the r highest row scores (default, 0).
                                 FVAR_SELECT_SAMPLE: r rows drawn without replacement with probability
                                 proportional to the row score (the sampling reading of Sec. 3.3 RTR): the r
                                 largest keys s_i / E_i, E_i ~ Exp(1) given in sample_noise                     */
  const float *sample_noise;  /* dev fp32 [n_groups][B_eff][M] of Exp(1) variates (> 0) for FVAR_SELECT_SAMPLE     */
  int restore;                /* how the M rows come back from the r rows of a FVAR_LOWRANK_RTR step.
                                 FVAR_RESTORE_RTR (default, 0): representative token restoration, the method
                                 (Sec. 3.3 RTR).  FVAR_RESTORE_LLS: the least-squares restoration the paper tries first
                                 (Sec. 3.3 RP, Eq. "lstsq"; App. A.3; Tab. "lowrank" row 5): F_k^o = (W_hat + W^{o,cache})
                                 F_r^o, W_hat the least-squares map from Q^T F back to the group's input F, W^{o,cache}
                                 the same for the upsampled cached group output (this library's reading: its r-row
                                 feature is its projection by the same Q).  No index set is chosen; r <= 192 per
                                 group (FVAR_EUNSUPPORTED beyond) and r <= the tokens of the cached scale (FVAR_EINVAL);
                                 a group's output then has rank r, so the next group should use a smaller r.  fp32 arithmetic; a Gram matrix that is not
                                 positive definite is reported as FVAR_EINVAL by fvar_poll_status.                  */
} fvar_keep_policy;

/* Bytes of device workspace fvar_init needs for this shape (0 if the shape is invalid). */
size_t fvar_workspace_bytes(const fvar_cfg *cfg);

/* Create a context.  `workspace` (dev, 1024-byte aligned, >= fvar_workspace_bytes) holds the KV
 * cache, the block-group output caches, projection matrices, index lists, activations and the
 * status word; it is zeroed here (enqueued on `cuda_stream`, a cudaStream_t passed as void*).
 * Builds the TMA descriptors of the weights.  FVAR_EINVAL / FVAR_EUNSUPPORTED on a bad shape,
 * FVAR_ENOMEM if `bytes` is too small, FVAR_ECUDA if no sm_100 device is current. */
fvar_status fvar_init(const fvar_weights *weights, const fvar_cfg *cfg, void *workspace, size_t bytes,
                      void *cuda_stream, fvar_ctx **out);

/* Hoisted conditioning (constant across scales): AdaLN vectors W_ada SiLU(c_b) + b_ada for every
 * block and batch element, and the cross-attention keys/values of the context tokens.  Also empties
 * the KV cache (a new generation starts).  cond dev bf16 [B][C]; context dev bf16
 * [B][ctx_len][ctx_width] or NULL without cross-attention.  B <= max_batch. */
fvar_status fvar_set_cond(fvar_ctx *ctx, int B, const void *cond, const void *context);

/* Random-projection matrix Q of Sec. 3.3 (entries N(0, 1/r)) for one (scale, block group), given
 * TRANSPOSED: Qt dev bf16 [r][M].  Copied into the workspace; shared by the whole batch.  Must be
 * set before a FVAR_LOWRANK_RTR step whose group rank is r < M. */
fvar_status fvar_set_projection(fvar_ctx *ctx, int scale_idx, int group, const void *Qt, int r);

/* The same matrix drawn on the device from a 64-bit seed instead of given (Sec. 3.3 RP: Q_ij ~
 * N(0, 1/r); the paper redraws Q per generation).  Generator: Philox4x32-10 (Salmon et al., SC'11);
 * call t with counter (t, group, scale_idx, 0) and key (seed low word, seed high word) yields elements
 * 4t .. 4t + 3 of Q^T flattened row-major (element j * M + i is Q_ij); uniforms u = (x + 0.5) 2^-32;
 * Box-Muller on the word pairs (0, 1) and (2, 3) in fp64: z = sqrt(-2 ln u_a) (cos, sin)(2 pi u_b);
 * Q = z / sqrt(r), rounded once to bf16.  Replaces any projection stored for (scale, group).
 * FVAR_EINVAL unless 0 < r <= M. */
fvar_status fvar_generate_projection(fvar_ctx *ctx, int scale_idx, int group, int r, unsigned long long seed);

/* Copies the stored projection of (scale, group), transposed as it was given or drawn, to
 * Qt_out dev bf16 [r][M] (asynchronous on the context's stream) and its rank to *r_host.
 * FVAR_ESTATE if none is stored. */
fvar_status fvar_get_projection(fvar_ctx *ctx, int scale_idx, int group, void *Qt_out, int *r_host);

/* Codebook Z (V codewords of width d) of the quantizer Q that Algorithm 1 lists among its inputs:
 * Z dev bf16 [V][C], 16-byte aligned, 1 <= V <= 65536, d = C (the block width).  The
 * library keeps the pointer (the caller keeps the memory alive) and computes |Z_v|^2 / 2 into its workspace.
 * FVAR_EUNSUPPORTED for a larger codebook. */
fvar_status fvar_set_codebook(fvar_ctx *ctx, const void *Z, int V);

/* The transition between two scale steps (Algorithm 1, the three lines after the blocks in both stages;
 * Eq. "var_upf", Eq. "var_downf"):
 *     R_k = Q(F_k^o);   F_k = F_{k-1} + Up(R_k, (h_K, w_K));   next input = Down(F_k, (h_{k+1}, w_{k+1})).
 * The paper leaves Q, Up and Down abstract; here Q takes the nearest codeword of every token in Euclidean
 * distance (arg-max of F_k^o Z^T - |Z_v|^2 / 2, decided on fp32 scores, lowest code on ties), Up is the
 * library's bilinear upsampling (as in the restoration fill) and Down averages the cells of the last
 * scale's grid that each target cell covers ("area" resampling).  F_0 = 0: scale 0 overwrites the map.
 * fo dev bf16 [B][M_k][C] (what fvar_scale_step returned for scale_idx, B = its B_eff), 16-byte aligned;
 * codes dev int32 [B][M_k] or NULL; next_tokens dev bf16 [B][M_{k+1}][C], or NULL when no further step follows
 * (always at the last scale; also when the remaining steps are skipped, Sec. 4.1: F_k, already at the final
 * resolution, is then the output).  Scales must come in order from 0 with one B (FVAR_ESTATE otherwise).  Asynchronous on the
 * context's stream; allocates nothing. */
fvar_status fvar_scale_transition(fvar_ctx *ctx, const void *fo, int scale_idx, int B, int *codes, void *next_tokens);

/* The same transition with the next step's tokens written for both branches of every CFG pair: next_tokens_pairs
 * dev bf16 [2 B][M_{k+1}][C], elements 2p and 2p + 1 both hold the tokens of image p (fo and codes as above, one
 * row set per image).  What a closed generation loop needs while the next step still runs both branches. */
fvar_status fvar_scale_transition_pairs(fvar_ctx *ctx, const void *fo, int scale_idx, int B, int *codes,
                                        void *next_tokens_pairs);

/* Classifier-free guidance on the outputs of a step that ran both branches: out[p] = null + guidance *
 * (prompt - null) for the CFG pair p = elements (2p, 2p + 1) = (prompt, null prompt) of `pair`.  The paper
 * only states that VAR combines the prompt and null-prompt branches by classifier-free guidance and that
 * a guidance of 0 leaves the null-prompt branch alone (Sec. 3.2, Sec. 3.3); applying it to the block
 * outputs is this library's reading.  pair dev bf16 [B][per_elem], B even, per_elem % 8 == 0; out dev bf16
 * [B / 2][per_elem]; both 16-byte aligned. */
fvar_status fvar_cfg_combine(const void *pair, int B, long long per_elem, float guidance, void *out, void *stream);

/* Copies the accumulated map F_k of the last transition, fp32 [B][h_K * w_K][C], to F_out (device). */
fvar_status fvar_get_feature(fvar_ctx *ctx, float *F_out);

/* One scale step (Algorithm 1: the dense loop body, or the fidelity-refinement loop body RP -> blocks
 * -> RTR).  tokens dev bf16 [B][M][C] with M = h_k * w_k; out dev bf16 [B_eff][M][C], B_eff = B
 * (pair) or B/2 (null-only).  Stages this scale's K/V rows at the cache tail; they become visible
 * to later scales only after fvar_kv_append.  A group with r == M runs the dense path (Q = I).
 * FVAR_LOWRANK_RTR needs the previous stepped scale's group outputs (FVAR_ESTATE otherwise) and a
 * projection for every group with r < M.  FVAR_SKIP enqueues nothing.  scale_idx must not decrease
 * (FVAR_ESTATE); a FVAR_CFG_PAIR step after a FVAR_CFG_NULL_ONLY step is FVAR_ESTATE. */
fvar_status fvar_scale_step(fvar_ctx *ctx, const void *tokens, int scale_idx, const fvar_keep_policy *policy,
                            void *out);

/* Same step with HOST buffers: copies tokens host->dev, runs the step, copies out dev->host, and
 * synchronises the stream before returning.  Pinned host memory makes the copies asynchronous.
 * tokens_host is [B][M][C] as for fvar_scale_step; with FVAR_CFG_NULL_ONLY only the elements 2p + 1
 * that the step reads are uploaded (one strided copy). */
fvar_status fvar_scale_step_host(fvar_ctx *ctx, const void *tokens_host, int scale_idx,
                                 const fvar_keep_policy *policy, void *out_host);

/* The same with the copies taken off the step's stream: the upload runs on a stream of its own, the step on
 * the context's stream once its tokens have arrived, the download on a third stream once the step has
 * finished, through two staging slots each way inside the workspace.  Consecutive calls therefore overlap:
 * the tokens of call n + 1 go up and the result of call n - 1 comes down while step n computes.  Returns as
 * soon as everything is enqueued.  tokens_host must stay valid and unchanged, and out_host must not be read,
 * until fvar_host_sync returns; both should be pinned (pageable memory makes the copies synchronous).
 * The paper has no counterpart (it times whole generations on one GPU); this is the library's end-to-end
 * entry point. */
fvar_status fvar_scale_step_host_async(fvar_ctx *ctx, const void *tokens_host, int scale_idx,
                                       const fvar_keep_policy *policy, void *out_host);

/* Waits for every upload, step and download enqueued so far (host-blocking). */
fvar_status fvar_host_sync(fvar_ctx *ctx);

/* Commit the rows staged by the last step of `scale_idx` (O(1), host only).  FVAR_ESTATE if that
 * scale was not the last one stepped or was already appended. */
fvar_status fvar_kv_append(fvar_ctx *ctx, int scale_idx);

/* Row indices chosen by the last FVAR_LOWRANK_RTR step for `group`: copies [B_eff][r] int32 into
 * idx_dev (device to device, stream-ordered) and stores r in *count_host. */
fvar_status fvar_get_indices(fvar_ctx *ctx, int group, int *idx_dev, int *count_host);

/* fp32 output of block group `group` at the last stepped scale: [B][M][C] floats copied to out_dev
 * (rows of batch elements the step did not compute are unspecified). */
fvar_status fvar_get_group_output(fvar_ctx *ctx, int group, float *out_dev);

/* Stand-ins for earlier scales (tests, benchmarks): load committed K/V rows, K and V dev bf16
 * [n_blocks][B][L][C], as the cache contents (cache length becomes L for every block), and load
 * block-group outputs dev fp32 [n_groups][B][M][C] as those of scale `scale_idx`. */
fvar_status fvar_load_kv(fvar_ctx *ctx, const void *K, const void *V, int L);
fvar_status fvar_load_group_cache(fvar_ctx *ctx, int scale_idx, const float *cache);

/* Returns to the state the last fvar_load_kv and fvar_load_group_cache established (cache lengths,
 * group outputs, last stepped scale), so that the late scales can be run again, e.g. under another
 * policy.  O(1), host only; the loaded group outputs are kept in a slot of their own that steps never
 * overwrite.  FVAR_ESTATE if nothing was loaded. */
fvar_status fvar_restore_loaded(fvar_ctx *ctx);

/* Options.  FVAR_OPT_CUDA_GRAPHS (default 1): fvar_scale_step captures the chain of launches between
 * its input and output conversions into a CUDA graph the first time it sees a combination of scale,
 * ranks, cache lengths and batch, and replays the graph afterwards (the launches only touch the
 * workspace).  Instantiating a graph is the one place where the CUDA driver may allocate memory on the
 * library's behalf.  Steps with forced_indices or with profiling enabled are launched directly.
 * FVAR_OPT_GEMM_MAX_SPLITS (default 1; 1, 2 or 4): largest split-K factor the GEMM tile picker may use.
 * Partial tiles go through a scratch area of the workspace and are added in a fixed order, so results do
 * not depend on timing.  When allowed, the picker splits only reductions of K >= 4096 whose tiles would
 * leave more than half of the SMs idle.  Measured: +2 % on the Infinity-shaped late scales, -5 % on the
 * VAR-d16 ones, hence off by default.
 * FVAR_OPT_SKINNY_MAX_ROWS (default 512; 0 .. 512): cap on the rows R = B_eff * r up to which a GEMM of the
 * step may take one of the cluster-split forms (the library's own rule picks per GEMM: the weight-streaming form up
 * to 32 rows for wide outputs; 128 x 128 tiles with the same K split for outputs of at most 2048 features up to 256
 * rows, up to 512 with a reduction of 4096 or more).  In that
 * form the weights are the M side of the MMA and the K range of a 128-feature tile is spread over a
 * thread-block cluster that reduces through distributed shared memory; it is bound by reading the weights
 * once.  0 never uses it.
 * FVAR_OPT_WAIT_KCYCLES (default 0 = about half a second): budget, in thousands of clock cycles, of every
 * bounded wait inside the step's kernels; a wait that runs out sets FVAR_ETIMEOUT (fvar_poll_status). */
enum { FVAR_OPT_CUDA_GRAPHS = 0, FVAR_OPT_GEMM_MAX_SPLITS = 1, FVAR_OPT_SKINNY_MAX_ROWS = 2, FVAR_OPT_WAIT_KCYCLES = 3 };
fvar_status fvar_set_option(fvar_ctx *ctx, int option, int value);

/* Measurement aid: while enabled, every kernel launch of this context is bracketed by CUDA events on
 * the context's stream.  fvar_profile_read synchronises and sums, for one kernel class, the event
 * time, the number of launches and the algorithmic flops and bytes (minimum traffic: operands read
 * once, results written once) of the launches recorded since fvar_profile_enable(ctx, 1). */
enum { FVAR_KCLASS_GEMM = 0, FVAR_KCLASS_ATTENTION = 1, FVAR_KCLASS_LN = 2, FVAR_KCLASS_SCORE = 3,
       FVAR_KCLASS_SELECT = 4, FVAR_KCLASS_RTR_FILL = 5, FVAR_KCLASS_CONVERT = 6, FVAR_KCLASS_COUNT = 7 };
fvar_status fvar_profile_enable(fvar_ctx *ctx, int on);
fvar_status fvar_profile_read(fvar_ctx *ctx, int kclass, double *total_ms, long long *launches, double *flops,
                              double *bytes);
/* Per-launch event times (ms) of one kernel class in launch order: up to `capacity` values into ms_host;
 * *count_host receives the number of launches recorded. */
fvar_status fvar_profile_dump(fvar_ctx *ctx, int kclass, float *ms_host, int capacity, int *count_host);

/* Committed cache rows of `block` (host value). */
int fvar_cache_len(const fvar_ctx *ctx, int block);

/* Number of kernels the library has launched on this context since fvar_init (host counter). */
long long fvar_launch_count(const fvar_ctx *ctx);

/* Synchronises the stream, reads the device status word and clears it.  FVAR_OK, FVAR_ETIMEOUT,
 * FVAR_EINVAL (bad forced_indices) or FVAR_ECUDA.  After a timeout the results of the steps since the last
 * poll are invalid; the library clears its reduction counters and drops its captured graphs, and the context
 * can be used again.  ctx == NULL polls the status word of the kernel-level entry points on the current device. */
fvar_status fvar_poll_status(fvar_ctx *ctx);

/* Empties the KV cache and the group caches (host state only; device memory is not cleared). */
fvar_status fvar_reset(fvar_ctx *ctx);
void fvar_destroy(fvar_ctx *ctx);
/* Message of the last error on this context (or of the last failed fvar_init when ctx is NULL). */
const char *fvar_last_error(const fvar_ctx *ctx);

/* ---------------------------------------------------------------------------------------------
 * The method's schedule (host only; no context, no device): which scale steps run how, and the
 * rank r of every block group.
 * ------------------------------------------------------------------------------------------- */

/* Rank for a keep ratio: r = floor(keep_ratio * M + 0.5), clamped to [1, M] (what fvar_scale_step
 * uses when rank_per_group is NULL).  0 if M <= 0. */
int fvar_rank_from_keep_ratio(int M, float keep_ratio);

/* Rank that a rank ratio stands for.  Sec. 3.2, Eq. "low_rank_percent": a ratio is a fraction of
 * n = min(M, d), so r = floor(ratio * min(M, width) + 0.5), clamped to [1, M].  0 on a bad shape. */
int fvar_rank_from_table_ratio(int M, int width, double ratio);

/* App. A.1, the table of mean rank ratios at energy threshold alpha = 0.96: the entry of block chunk
 * `chunk` (0..7) at late scale `scale_side` (40, 48 or 64).  FVAR_EINVAL outside the table. */
fvar_status fvar_infinity_rank_ratio(int chunk, int scale_side, double *ratio_host);

/* Rank per block group at a late Infinity scale (40, 48 or 64 tokens a side, M = side^2) from that
 * table: ranks_host[g], g < n_groups.  With 8 groups, group g is chunk g; another group count takes
 * the chunk at the nearest relative depth (the paper prints the table for 8 chunks only). */
fvar_status fvar_infinity_group_ranks(int scale_side, int width, int n_groups, int *ranks_host);

/* The 13-step Infinity schedule of Sec. 4.1: side length and mode (FVAR_DENSE / FVAR_LOWRANK_RTR /
 * FVAR_SKIP) of every scale step.  Scales 1..32 are dense; 40, 48, 64 have thresholds alpha =
 * {0.96, 0, 0} and alpha = 0 skips the step (paper_schedule != 0), or all three are approximated
 * (paper_schedule == 0).  Writes min(13, capacity) entries to each non-NULL array, 13 to *count_host. */
fvar_status fvar_infinity_schedule(int paper_schedule, int capacity, int *sides_host, int *modes_host, int *count_host);

/* ---------------------------------------------------------------------------------------------
 * Kernel-level entry points: the individual steps of the path, callable on caller-owned device
 * buffers.  `stream` is a cudaStream_t passed as void*.  They synchronise nothing.
 * ------------------------------------------------------------------------------------------- */

/* Row score of Sec. 3.3 (RTR): s[b][i] = sum_c x[b][i][c]^2 (the numerator of p_i; the common
 * denominator ||X||_F^2 does not change the order).  x dev fp32 [B][M][C], C % 4 == 0; scores dev fp32 [B][M]. */
fvar_status fvar_row_scores(const float *x, int B, int M, int C, float *scores, void *stream);

/* Sampling keys of the row selection: keys[b][i] = s[b][i] / noise[b][i] (one fp32 division, round to
 * nearest) with s the row score above and noise dev fp32 [B][M] of Exp(1) variates.  Feeding the keys
 * to fvar_select_topr draws r rows without replacement with probability proportional to s (Sec. 3.3). */
fvar_status fvar_row_keys(const float *x, const float *noise, int B, int M, int C, float *keys, void *stream);

/* Index set I of Sec. 3.3 / Algorithm 1: per batch element the r highest-scoring rows, ascending.
 * Order: score descending then index ascending; NaN ranks as +inf; -0 == +0.
 * scores dev fp32 [B][M]; idx dev int32 [B][r]; inv dev int32 [B][M] (position j of row i in idx, or -1). */
fvar_status fvar_select_topr(const float *scores, int B, int M, int r, int *idx, int *inv, void *stream);

/* LayerNorm (no affine, biased variance) + AdaLN modulation: y = LN(x) * (1 + scale) + shift.
 * x dev fp32 [R][C]; shift/scale dev fp32, row i uses the vectors at offset (i / rows_per_batch) *
 * vec_stride floats; y dev bf16 [R][C].  C % 8 == 0, C <= 8192. */
fvar_status fvar_ln_modulate(const float *x, int R, int C, int rows_per_batch, const float *shift,
                             const float *scale, long long vec_stride, float eps, void *y, void *stream);

/* out[R][N] (fp32) = A[R][K] W[N][K]^T + bias[N] on the tensor cores (bf16 operands, fp32
 * accumulation).  A, W, bias dev bf16 (bias may be NULL); K % 8 == 0; lda = ldw = K. */
fvar_status fvar_gemm_bf16(const void *A, const void *W, const void *bias, int R, int N, int K, float *out,
                           void *stream);

/* The same product with the second operand given transposed: Wt dev bf16 [K][N] row-major (ldw = N, N % 8 == 0),
 * out = A Wt + bias.  The tensor core then reads W as an MN-major operand; nothing is transposed in memory.
 * block_n in {0 (picked), 64, 128, 256}; single-CTA tiles.  Used by the random projection F_r = Q^T F (Sec. 3.3 RP),
 * whose second operand, the token rows, is stored [M][C]. */
fvar_status fvar_gemm_bf16_wt(const void *A, const void *Wt, const void *bias, int R, int N, int K, int block_n,
                              float *out, void *stream);

/* The same product with the launch form given instead of picked: form FVAR_GEMM_AUTO (the library's
 * cost model, as fvar_gemm_bf16), FVAR_GEMM_SINGLE (one CTA per 128 x block_n tile, block_n in
 * {64, 128, 256}) or FVAR_GEMM_PAIR (two CTAs on neighbouring SMs share one 256 x block_n tile through
 * tcgen05.mma.cta_group::2, block_n in {128, 256}; needs R > 128).  block_n = 0 lets the cost model
 * pick the width for the given form.  The transformer block of the step is the workload's own
 * definition (the paper only names it a "VAR block", Sec. 3.1), so this is a kernel-level entry for
 * tests and tuning.  FVAR_GEMM_SKINNY: the weight-streaming form for R <= 512 (see FVAR_OPT_SKINNY_MAX_ROWS);
 * block_n is then the number of K ranges per 128-feature tile, 1 .. 8, or 0 to let the library pick.  FVAR_GEMM_KSPLIT:
 * 128 x 128 output tiles (rows on the M side, any R) whose K range is spread over a cluster in the same way.
 * FVAR_EINVAL for a form / width the problem does not allow. */
#define FVAR_GEMM_AUTO 0
#define FVAR_GEMM_SINGLE 1
#define FVAR_GEMM_PAIR 2
#define FVAR_GEMM_SKINNY 3
#define FVAR_GEMM_KSPLIT 4
fvar_status fvar_gemm_bf16_form(const void *A, const void *W, const void *bias, int R, int N, int K, int form,
                                int block_n, float *out, void *stream);

/* softmax(q k^T / sqrt(D)) v per head over the first L rows of a cache in the library's layout:
 * q dev bf16 [B][r][H*D]; Kc dev bf16 [B][H][L_cap][D]; Vt dev bf16 [B][H][D][L_cap] (values stored
 * transposed); out dev bf16 [B][r][H*D].  D in {64, 128}; L_cap % 8 == 0; 1 <= L <= L_cap. */
fvar_status fvar_attention(const void *q, const void *Kc, const void *Vt, int B, int H, int r, int D, int L,
                           int L_cap, void *out, void *stream);

/* Failure-detection self-test: launches one CTA that waits, with a budget of `cycles` clock cycles, on a
 * barrier nothing ever signals.  The wait gives up, the kernel records FVAR_ETIMEOUT in the status word and
 * returns; nothing faults or hangs.  The next fvar_poll_status(ctx) returns FVAR_ETIMEOUT, the one after
 * FVAR_OK.  ctx == NULL uses the kernel-level status word and `stream`.  The paper has no counterpart. */
fvar_status fvar_selftest_wait_timeout(fvar_ctx *ctx, long long cycles, void *stream);

/* Asks the L2 cache to fetch [ptr, ptr + bytes) (ptr dev, 16-byte aligned; bytes rounded down to a multiple of
 * 16): a hint for data a later kernel will stream, e.g. the weights of the next layer while the current one
 * computes.  The range must not be written by work still in flight on the stream.  The paper has no
 * counterpart (it describes no kernels); the step uses the same hint between its GEMMs. */
fvar_status fvar_l2_prefetch(const void *ptr, size_t bytes, void *stream);

/* Restoration fill of Eq. "redefine" with Eq. "upcache": for every row i of batch element b with
 * inv[b][i] < 0, out[b][i] = Up(prev[b])[i], bilinear with half-pixel centres on the (h, w) grid.
 * prev dev fp32 [B][h0*w0][C]; out dev fp32 [B][h1*w1][C]; rows with inv >= 0 are left untouched;
 * inv == NULL fills every row.  C % 4 == 0. */
fvar_status fvar_rtr_fill(const float *prev, int B, int h0, int w0, int h1, int w1, int C, const int *inv,
                          float *out, void *stream);

/* Row selection for callers that cannot allocate device memory (the paper has no counterpart: this
 * is a packaging variant of fvar_row_scores followed by fvar_select_topr, same results bit for bit).
 * Who needs it: code that runs inside someone else's memory plan -- an inference server that
 * reserves all of HBM at start-up, a plugin under another framework's allocator, a real-time loop
 * where cudaMalloc's implicit synchronisation is not acceptable -- and so has nowhere to put the
 * [B][M] scores that sit between the two kernels.  Here they live in a fixed fp32 array inside the
 * library image: FVAR_STATIC_SELECT_MAX_ROWS entries (256 KiB), resident on every GPU that loads
 * the library until the process exits.  The call allocates and frees nothing.
 *   x dev fp32 [B][M][C] (C % 4 == 0); idx dev int32 [B][r]; inv dev int32 [B][M]; both written in full.
 *   B * M > FVAR_STATIC_SELECT_MAX_ROWS -> FVAR_EUNSUPPORTED with a message (use the two-call form).
 * The first call on each device looks up the array's device address (cudaGetSymbolAddress, with
 * that device current); make that first call before starting any stream capture.  All calls on a
 * device share the one array, which simply keeps the previous call's scores: every entry a call
 * reads it has just written, so nothing needs clearing -- but two calls whose kernels can overlap
 * on the GPU (different streams without an ordering between them) race on it; serialise them. */
#define FVAR_STATIC_SELECT_MAX_ROWS 65536
fvar_status fvar_select_rows_static(const float *x, int B, int M, int C, int r, int *idx, int *inv, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* FVAR_H_ */
