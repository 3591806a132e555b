/*
 * cb.h - C ABI of the head-local KV-cache mapper construction and apply library (CUDA, sm_100a).
 *
 * The library builds, for every target (component, layer l, KV head h) matched to ONE source head
 * (layer j(l), head a(h)), the attention-weighted sufficient statistics of an affine ridge map, solves the
 * ridge systems in closed form, and applies the fitted maps to a source cache.
 *
 * Notation (paper, Section 2.1): source model L_s layers, H_s KV heads, head width d_s; target L_t, H_t, d_t.
 * comp = 0 for keys, 1 for values.  Map id  m = (comp*L_t + l)*H_t + h,  n_maps = 2*L_t*H_t.
 * d = d_s = d_t, p = d + 1.  Row-vector convention y_hat = x W + b (Section 3.1); the bias is the LAST row of
 * Theta = [W; b] and the LAST row/column of G.
 *
 * All device pointers are plain CUDA device pointers owned by the caller.  The library allocates no device
 * memory.  Every call enqueues its work on the given stream (a cudaStream_t passed as void*, NULL = default
 * stream) and returns without synchronising unless stated.  Errors are returned as status codes; argument
 * errors are detected on the host before anything is launched.  Preconditions that are NOT checked on the
 * device: weights are finite and >= 0, traces are finite.
 *
 * There is no CPU implementation behind these calls: without a CUDA device they return CB_ERR_CUDA.
 */
#ifndef CB_H_
#define CB_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum cb_status {
    CB_OK = 0,
    CB_ERR_INVALID_ARG = 1,  /* null pointer, negative size, stride not usable, misaligned pointer        */
    CB_ERR_UNSUPPORTED = 2,  /* head width not in {64, 128}, d_s != d_t, too many tokens in one call       */
    CB_ERR_STATE = 3,        /* call order violated (e.g. reduce before any accumulate is fine, but a      */
                             /* destroyed or foreign context is not)                                       */
    CB_ERR_WORKSPACE = 4,    /* workspace smaller than cb_workspace_bytes() or not 256-byte aligned         */
    CB_ERR_CUDA = 5,         /* a CUDA runtime/driver call failed (includes "no device")                    */
    CB_ERR_NOT_PD = 6,       /* cb_check_info: at least one ridge system had a non-positive pivot           */
    CB_ERR_TIMEOUT = 7,      /* cb_device_status / cb_last_device_status: a bounded device-side wait ran out */
    CB_ERR_STATIC_LIMIT = 8  /* cb_stats_build_static: the problem needs more scratch than the built-in buffer  */
} cb_status;

/* flags (cb_problem.flags and the flags argument of cb_ridge_solve) */
#define CB_FLAG_COMPENSATED 1u /* accumulate: split the bf16 weighted operand into hi + lo (two MMAs per   */
                               /* tile) so that folding the fp32 weight into a bf16 operand costs ~2^-17   */
                               /* instead of ~2^-9 per element.  Meant for small token counts; calls of     */
                               /* fewer than 4,096 rows use it in any case.                                 */
#define CB_FLAG_RAW_LAMBDA  2u /* solve: penalise with lambda itself instead of lambda * s_w / n            */
#define CB_FLAG_SIMT        4u /* accumulate/apply: use the plain fp32 CUDA-core kernels (no tensor cores) */
#define CB_FLAG_ONE_ROW_HEAD 8u /* cb_fullhead_problem only: statistics by the kernel that weights one feature head  */
                               /* per unit (three staged tiles for two products) instead of the default 2 x 2 blocked */
                               /* kernel (four tiles for four products); kept as a cross-check                        */

#define CB_DTYPE_BF16 0
#define CB_DTYPE_F32  1

/*
 * A strided bf16 view of one model's K and V traces (or caches) for n_tokens rows; device memory.
 * Element (layer j, token t, head g, channel c) of K is at
 *     (bf16*)k + j*stride_layer + t*stride_token + g*stride_head + c          (strides in elements)
 * and likewise for V.  Channels are contiguous.  This covers the paper's index order K_{j,t,g} stored as
 * [L][T][H][d] as well as [L][H][T][d].  k and v must be 16-byte aligned and every stride a multiple of 8.
 * A stride of 0 (a broadcast view, e.g. one head expanded to several) is accepted only on a dimension of size 1;
 * otherwise the call returns CB_ERR_UNSUPPORTED.  The same holds for the output strides of the apply calls.
 */
typedef struct cb_kv_view {
    const void *k;
    const void *v;
    int32_t n_layers, n_heads, head_dim;
    int64_t n_tokens;
    int64_t stride_layer, stride_token, stride_head;
} cb_kv_view;

/*
 * The mapping problem: model shapes and the static head match (Section 3.2, Eq. "localfeature" with one
 * selected layer per target layer): target layer l reads source layer src_layer[l]; target head h reads
 * source head src_head[h].  src_layer (length Lt) and src_head (length Ht) are HOST arrays, copied by
 * cb_create / read by cb_apply during the call.
 * n_splits: number of token splits (independent partial statistics per map, summed in fixed order by
 * cb_stats_reduce); 0 lets the library choose (cb_token_splits reports the choice, which depends on the
 * problem's shapes only).  Must be <= 64.
 */
typedef struct cb_problem {
    int32_t Ls, Hs, ds;
    int32_t Lt, Ht, dt;
    const int32_t *src_layer;
    const int32_t *src_head;
    uint32_t flags;
    int32_t n_splits;
} cb_problem;

typedef struct cb_ctx cb_ctx;

const char *cb_status_string(cb_status s);

/*
 * Default head match.  Layer: nearest relative depth, j(l) = floor((2 l (Ls-1) + (Lt-1)) / (2 (Lt-1)))
 * (0 if Lt == 1); head: a(h) = floor(h*Hs/Ht), the identity when both models expose the same number of KV
 * groups (Section 3.2).  Host arrays of length Lt and Ht.
 */
cb_status cb_head_map_nearest(int32_t Ls, int32_t Hs, int32_t Lt, int32_t Ht,
                              int32_t *src_layer, int32_t *src_head);

/*
 * Static gather schedule (Section 2.3: support and head assignment are fixed before fitting, so the irregular
 * gather is compiled once).  Maps are grouped by the source head they read.  Items are ordered by
 * (comp, source layer, source head); only source heads read by at least one map become items; the maps of an
 * item are listed in ascending id.  Host output arrays: item_comp/item_layer/item_head need 2*Ls*Hs entries,
 * item_begin 2*Ls*Hs + 1 (offsets into item_maps), item_maps 2*Lt*Ht.  *n_items receives the item count.
 */
cb_status cb_work_list(const cb_problem *prob, int32_t *n_items, int32_t *item_comp, int32_t *item_layer,
                       int32_t *item_head, int32_t *item_begin, int32_t *item_maps);

/* Bytes of device workspace cb_create needs for this problem (partial statistics slots + small tables). */
cb_status cb_workspace_bytes(const cb_problem *prob, size_t *bytes);

/*
 * The number of token splits the statistics calls will use for this problem (Section 3.4: partial statistics
 * per bounded block of observations, then a fixed reduction): prob->n_splits if it is positive, else the count in
 * 1..8 that balances the persistent blocks' units (map, split) over the current device's SMs (148 if there is no
 * device to ask) against the cost of one more set of partial slots per split.  Host only; *n_splits receives the count.
 */
cb_status cb_token_splits(const cb_problem *prob, int32_t *n_splits);

/*
 * Create a context on the current device.  workspace: device memory, 256-byte aligned, at least
 * cb_workspace_bytes(); it stays owned by the caller and must outlive the context.  Copies the head match
 * to the device (synchronous, small) and leaves the statistics in the reset state (zero) by enqueueing a
 * clear on the default stream and synchronising it.
 */
cb_status cb_create(const cb_problem *prob, void *workspace, size_t workspace_bytes, cb_ctx **out);
void cb_destroy(cb_ctx *ctx);

/* Zero the partial statistics and the token count. */
cb_status cb_stats_reset(cb_ctx *ctx, void *stream);

/*
 * Fused weighted-statistics accumulation (Section 3.4, Eq. "fusedstats", in the bias-column form): for every
 * map m with matched source head, add over the n_tokens rows of this call
 *     G_m += sum_t w_t [x_t,1]^T [x_t,1]      C_m += sum_t w_t [x_t,1]^T y_t
 * reading x_t from src (layer src_layer[l], head src_head[h]), y_t from tgt (layer l, head h) and
 * w_t from w_k (keys) or w_v (values) at  w + l*w_stride_layer + h*w_stride_head + t  (fp32, device,
 * strides in elements, tokens contiguous).  w_v may equal w_k.  No concatenated observation matrix is built;
 * head pairs are read straight from the strided views.  Statistics are additive over calls (token chunks of
 * any size, including ragged batches packed back to back); src->n_tokens must equal tgt->n_tokens and be
 * < 2^31.  n_tokens == 0 is a no-op.  Partial sums live in fp32 in the context's workspace: each (map, split)
 * slot is owned by one thread block per call and calls are ordered by the stream, so results are bitwise
 * reproducible for a fixed sequence of calls.
 */
cb_status cb_stats_accumulate(cb_ctx *ctx, const cb_kv_view *src, const cb_kv_view *tgt,
                              const float *w_k, const float *w_v,
                              int64_t w_stride_layer, int64_t w_stride_head, void *stream);

/*
 * The same accumulation for a chunk that lives in HOST memory (the end-to-end path of a streaming build whose
 * traces do not fit on the device).  src/tgt are views of host memory and must be dense in the order
 * [layer][token][head][channel] (stride_head = d, stride_token = H*d, stride_layer = n_tokens*H*d); w_k / w_v are
 * host fp32 [Lt][Ht][n_tokens] dense.  staging is caller-owned DEVICE memory of at least
 * cb_staging_bytes(prob, n_tokens) bytes, 256-byte aligned.  The call enqueues the host-to-device copies and then
 * the accumulation on the stream; the host buffers (pinned memory gives asynchronous copies) and the staging
 * buffer must stay untouched until that work has completed.
 */
cb_status cb_staging_bytes(const cb_problem *prob, int64_t n_tokens, size_t *bytes);
cb_status cb_stats_accumulate_host(cb_ctx *ctx, const cb_kv_view *src_host, const cb_kv_view *tgt_host,
                                   const float *w_k_host, const float *w_v_host,
                                   void *staging, size_t staging_bytes, void *stream);

/*
 * Deterministic reduction: sums the splits of every map in index order (fp64 inside), symmetrises
 * G <- (G + G^T)/2 and writes fp32  G [n_maps][p][p]  and  C [n_maps][p][d]  (device).  n_tokens_out (host,
 * may be NULL) receives the number of rows accumulated since the last reset; it is host bookkeeping and
 * valid on return.  The partial statistics are left untouched, so accumulation can continue afterwards.
 */
cb_status cb_stats_reduce(cb_ctx *ctx, float *G, float *C, int64_t *n_tokens_out, void *stream);

/*
 * Checkpoint and resume of a streamed build (Section 3.4: statistics are sums over bounded blocks of observations, so
 * the partial statistics ARE the state of the build).  cb_stats_export copies the partial slots of the context
 * (cb_stats_state_bytes() bytes, fp32) to `dst`, device or host memory, on the stream and returns the number of rows
 * accumulated so far; cb_stats_import replaces the context's state by such a copy (same problem shapes and the same
 * number of token splits: the byte count must match, CB_ERR_INVALID_ARG otherwise) and sets the row count.
 * Accumulation continues bit-identically after an import.  For the one-pass statistics; a two-pass build checkpoints
 * its means workspace and mu the same way (they are plain caller-owned buffers).
 */
cb_status cb_stats_state_bytes(cb_ctx *ctx, size_t *bytes);
cb_status cb_stats_export(cb_ctx *ctx, void *dst, size_t dst_bytes, int64_t *n_tokens_out, void *stream);
cb_status cb_stats_import(cb_ctx *ctx, const void *src, size_t src_bytes, int64_t n_tokens, void *stream);

/*
 * Batched closed-form ridge solve (Section 3.1, Eq. "closedform", written for the bias-column statistics):
 * for every lambda and map,  (G_m + lambda_eff J) Theta = C_m,  J = diag(1,..,1,0) (bias not penalised),
 * by Cholesky factorisation in fp64.  lambda_eff = lambda * s_w / n_tokens with s_w = G_m[d][d] (the paper
 * states the objective for weights rescaled to mean one; this is that rescale), or lambda itself with
 * CB_FLAG_RAW_LAMBDA.  G [n_maps][p][p], C [n_maps][p][d]: device fp32.  lambdas: HOST array of n_lambda
 * (<= 16) values.  Wb: device fp32 [n_lambda][n_maps][p][d] (rows 0..d-1 = W, row d = b).  info: device int32
 * [n_lambda][n_maps]: 0, or r > 0 if pivot r was not positive, in which case that map's Wb is zero-filled.
 */
cb_status cb_ridge_solve(const float *G, const float *C, int32_t n_maps, int32_t d, int64_t n_tokens,
                         const float *lambdas, int32_t n_lambda, uint32_t flags,
                         float *Wb, int32_t *info, void *stream);

/*
 * The same solve for wider regressors (head-local support over k > 1 selected layers, Section 3.2: P = k*d + 1, e.g.
 * 1025 for k = 8), where a system does not fit in shared memory: blocked Cholesky and substitutions in fp64 on a
 * padded copy of every system.  G [n_maps][P][P], C [n_maps][P][d], Wb [n_lambda][n_maps][P][d], info as above.
 * workspace: device, 256-byte aligned, at least cb_ridge_solve_large_workspace_bytes(P, d, 1); systems are processed
 * in batches of as many as fit (all n_lambda * n_maps at once if the workspace is large enough).
 */
cb_status cb_ridge_solve_large_workspace_bytes(int32_t P, int32_t d, int64_t n_systems, size_t *bytes);
cb_status cb_ridge_solve_large(const float *G, const float *C, int32_t n_maps, int32_t P, int32_t d, int64_t n_tokens,
                               const float *lambdas, int32_t n_lambda, uint32_t flags,
                               float *Wb, int32_t *info, void *workspace, size_t workspace_bytes, void *stream);

/* Synchronises the stream and returns CB_ERR_NOT_PD if any of the n info entries is non-zero
 * (*first_bad, may be NULL, receives its index), CB_OK otherwise. */
cb_status cb_check_info(const int32_t *info, int64_t n, void *stream, int64_t *first_bad);

/*
 * Online affine apply (Section 3.2; Section 1, online handoff): for every map m and token t of the source
 * cache,  out[l][t][h][:] = x_t W_m + b_m  with x_t the matched source head's row.  Wb: device fp32
 * [n_maps][p][d].  Outputs tgt_k / tgt_v: device, element (l, t, h, c) at
 * l*t_stride_layer + t*t_stride_token + h*t_stride_head + c (elements of out_dtype: CB_DTYPE_BF16 rounds to
 * nearest even, CB_DTYPE_F32 stores fp32), 16-byte aligned, strides multiples of 8.  Positional rotation is
 * the caller's: the map acts in content coordinates.  prob->flags & CB_FLAG_SIMT selects the CUDA-core kernel.
 */
cb_status cb_apply(const cb_problem *prob, const float *Wb, const cb_kv_view *src_cache,
                   void *tgt_k, void *tgt_v, int64_t t_stride_layer, int64_t t_stride_token,
                   int64_t t_stride_head, int32_t out_dtype, void *stream);

/*
 * Effective-sample-size floor on the calibration weights (Section 3.3): for each of the n_rows rows (one per layer,
 * head and component) of raw sensitivities r_raw >= 0 over n_tokens rows of the calibration set,
 *     r_i = r_raw_i / mean(r_raw),  CV^2 = mean (r_i - 1)^2,  tau = min(n, 2 p_width),
 *     alpha* = 1 if CV^2 = 0 else min(1, sqrt((n / tau - 1) / CV^2)),      w_i = 1 + alpha* (r_i - 1),
 * so that the Kish effective sample size n / (1 + alpha^2 CV^2) of the mean-one weights stays >= tau.
 * r_raw, w: device fp32, row r at base + r*row_stride (elements), may not overlap; alpha_out: device fp32 [n_rows]
 * or NULL.  p_width is the regressor's feature width (k * d_s).  A row without any sensitivity gives w = 1.
 * The whole calibration set of a row must be passed in one call (the floor depends on n).
 */
cb_status cb_ess_weights(const float *r_raw, int32_t n_rows, int64_t n_tokens, int64_t r_row_stride,
                         int64_t p_width, float *w, int64_t w_row_stride, float *alpha_out, void *stream);

/*
 * Full-head contrast (Section 3.1, Eq. "fullheadfeature"; the inherited baseline of Section 2.1): every target head
 * of layer l is regressed from ALL H_s source KV heads of k selected source layers, feature order layer-major, then
 * head, then channel, bias last: P_f = k*H_s*d + 1.  Statistics per (comp, l): one G (P_f x P_f) shared by the
 * layer's heads and one C (P_f x d) per target head; the weights are per (comp, l, token).
 *
 * cb_fullhead_layer_sets: default selection, k consecutive source layers starting one below the nearest-depth layer
 * j(l), shifted into [0, Ls-1] (host array [Lt][k]).
 * cb_fullhead_stats_accumulate ADDS the statistics of this call's n_tokens rows to
 *     G [2][Lt][P_f][P_f]   and   C [2][Lt][Ht][P_f][d]        (device fp32, caller-owned, zeroed by the caller
 * before the first call).  G is filled on both triangles and is exactly symmetric (the call ends by copying the
 * lower triangle over the upper one; with CB_FLAG_ONE_ROW_HEAD the d x d diagonal blocks are left as computed).
 * w_k / w_v: device fp32 [Lt][n_tokens] at w + l*w_stride_layer + t.  layer_sets: HOST [Lt][k], ascending layers in
 * [0, Ls-1]; k*Hs <= 64 (an odd number of feature heads is fine).  workspace: device, 256-byte aligned,
 * cb_fullhead_workspace_bytes() (small index tables, copied inside the call).  Same stream/ownership/error rules as
 * cb_stats_accumulate; no context.
 */
typedef struct cb_fullhead_problem {
    int32_t Ls, Hs, ds;
    int32_t Lt, Ht, dt;
    int32_t k;
    const int32_t *layer_sets;
    uint32_t flags;
} cb_fullhead_problem;
cb_status cb_fullhead_layer_sets(int32_t Ls, int32_t Lt, int32_t k, int32_t *layer_sets);
cb_status cb_fullhead_workspace_bytes(const cb_fullhead_problem *prob, size_t *bytes);
cb_status cb_fullhead_stats_accumulate(const cb_fullhead_problem *prob, const cb_kv_view *src, const cb_kv_view *tgt,
                                       const float *w_k, const float *w_v, int64_t w_stride_layer,
                                       float *G, float *C, void *workspace, size_t workspace_bytes, void *stream);

/*
 * Head-local support over k > 1 selected source layers (Section 3.2, Eq. "localfeature": the paper's operating point,
 * k = 8 for Qwen3): the feature of target (l, h) concatenates source head src_head[h] of the k layers
 * prob->layer_sets[l][0..k-1] (layer-major, bias last), P = k*d + 1.  cb_multilayer_stats_accumulate ADDS this call's
 * statistics to G [n_maps][P][P] and C [n_maps][P][d] (device fp32, caller-owned, zeroed by the caller first; map id
 * m = (comp*Lt + l)*Ht + h; both triangles of G are filled).  Weights per (comp, l, h, token) as for
 * cb_stats_accumulate.  prob->Hs, prob->Ht describe the models; src_head: HOST [Ht].  workspace: device, 256-byte
 * aligned, cb_multilayer_workspace_bytes().  The systems are solved with cb_ridge_solve_large.
 */
cb_status cb_multilayer_workspace_bytes(const cb_fullhead_problem *prob, size_t *bytes);
cb_status cb_multilayer_stats_accumulate(const cb_fullhead_problem *prob, const int32_t *src_head,
                                         const cb_kv_view *src, const cb_kv_view *tgt,
                                         const float *w_k, const float *w_v, int64_t w_stride_layer, int64_t w_stride_head,
                                         float *G, float *C, void *workspace, size_t workspace_bytes, void *stream);

/*
 * Online apply for the same support:  out[l][t][h][:] = sum_f x_f W_f + b  with x_f the row of source head src_head[h]
 * of layer layer_sets[l][f] and W_f the f-th d x d block of the map's Wb [n_maps][k*d + 1][d] (bias row last).
 * Outputs and strides as for cb_apply.  workspace: device, 256-byte aligned, cb_apply_multilayer_workspace_bytes()
 * (the bf16 hi/lo image of all maps, rebuilt by every call).
 */
cb_status cb_apply_multilayer_workspace_bytes(const cb_fullhead_problem *prob, size_t *bytes);
cb_status cb_apply_multilayer(const cb_fullhead_problem *prob, const int32_t *src_head, const float *Wb,
                              const cb_kv_view *src_cache, void *tgt_k, void *tgt_v,
                              int64_t t_stride_layer, int64_t t_stride_token, int64_t t_stride_head, int32_t out_dtype,
                              void *workspace, size_t workspace_bytes, void *stream);

/* ------------------------------------------------------------------------------------------------------------------
 * Two-pass centred construction (Section 3.4, Eq. "fusedstats" and the solve displayed below it).
 *
 * The paper's own construction: a first pass obtains the weighted means of every map by a fixed reduction tree,
 * a second pass accumulates the centred statistics
 *     A = sum_t w_t (x_t - mu_x)(x_t - mu_x)^T   [d][d],      B = sum_t w_t (x_t - mu_x)(y_t - mu_y)^T   [d][d],
 * and the solve is  W = (A + lambda_eff I)^-1 B,  b = mu_y - mu_x W.  It is the same estimator as the one-pass
 * bias-column path above; it costs a second read of the traces and is the robust choice when channel means dwarf
 * the spread (the one-pass operand w x is rounded to bf16 BEFORE the mean cancels, the two-pass operand w (x - mu_x)
 * after).  Both passes are additive over calls, so a streamed build runs pass 1 over all chunks, finalises, then
 * pass 2 over all chunks.
 *
 * Call order:  cb_means_reset; cb_means_accumulate per chunk; cb_means_finalize -> mu;
 *              cb_stats_reset; cb_stats_accumulate_centered per chunk (same chunks, same mu);
 *              cb_stats_reduce_centered -> A, B;  cb_ridge_solve_centered -> Wb (same layout as cb_ridge_solve, so
 *              cb_apply consumes it unchanged).
 *
 * means_ws: caller-owned device memory, 256-byte aligned, at least cb_means_workspace_bytes() bytes (fp64 partial
 * sums of w x, w y, w and w y^2, 8 token splits per map); it carries the first-pass state between calls.
 * mu: device fp32 [n_maps][2 d + 1], per map  mu_x [d], mu_y [d], s_w  (a map whose weights sum to zero gets zero
 * means).  Reduction order is fixed (per thread in token order, row groups in index order, splits in index order,
 * chunks in call order), so results are bitwise reproducible for a fixed sequence of calls.
 * The accumulate call takes the same arguments as cb_stats_accumulate plus mu; it uses the context's partial slots
 * (do not mix one-pass and centred accumulation between two resets) and is not available with CB_FLAG_SIMT
 * (CB_ERR_UNSUPPORTED).  cb_stats_reduce_centered writes fp32 A [n_maps][d][d] (exactly symmetric) and
 * B [n_maps][d][d].  cb_ridge_solve_centered: arguments as cb_ridge_solve with (A, B, mu) in place of (G, C);
 * lambda_eff = lambda * s_w / n_tokens unless CB_FLAG_RAW_LAMBDA.
 * Errors: as for their one-pass counterparts; CB_ERR_WORKSPACE for a missing, misaligned or short means_ws.
 */
cb_status cb_means_workspace_bytes(const cb_problem *prob, size_t *bytes);
cb_status cb_means_reset(cb_ctx *ctx, void *means_ws, size_t means_ws_bytes, void *stream);
cb_status cb_means_accumulate(cb_ctx *ctx, const cb_kv_view *src, const cb_kv_view *tgt,
                              const float *w_k, const float *w_v, int64_t w_stride_layer, int64_t w_stride_head,
                              void *means_ws, size_t means_ws_bytes, void *stream);
cb_status cb_means_finalize(cb_ctx *ctx, const void *means_ws, size_t means_ws_bytes, float *mu, void *stream);
cb_status cb_stats_accumulate_centered(cb_ctx *ctx, const cb_kv_view *src, const cb_kv_view *tgt,
                                       const float *w_k, const float *w_v,
                                       int64_t w_stride_layer, int64_t w_stride_head, const float *mu, void *stream);
cb_status cb_stats_reduce_centered(cb_ctx *ctx, const float *mu, float *A, float *B, int64_t *n_tokens_out, void *stream);
cb_status cb_ridge_solve_centered(const float *A, const float *B, const float *mu, int32_t n_maps, int32_t d,
                                  int64_t n_tokens, const float *lambdas, int32_t n_lambda, uint32_t flags,
                                  float *Wb, int32_t *info, void *stream);

/* ------------------------------------------------------------------------------------------------------------------
 * Rotary position embedding at the boundary (Section 2.2; Section 3.1: source RoPE is inverted before fitting and
 * target RoPE applied after mapping, so the affine map acts in content coordinates).  Keys only: values carry no
 * rotary embedding and take the ordinary path.
 *
 * Convention (the paper prints none; this is the rotate-half form of the Llama / Qwen families): channel i < d/2
 * pairs with channel i + d/2, angle phi_i = position * base^(-2 i / d); the embedding maps (x_i, x_{i+d/2}) to
 * (x_i cos phi - x_{i+d/2} sin phi, x_i sin phi + x_{i+d/2} cos phi).  The whole head dimension rotates.
 * positions: DEVICE int32 [n_tokens], the position of every row (ragged batches: each sequence restarts at its own
 * origin), 4-byte aligned, 0 <= position < 2^20.  rope_base in (1, 1e12].
 *
 * cb_stats_accumulate_rope: as cb_stats_accumulate, but the key maps are fitted on source keys with the source
 * model's embedding removed and target keys with the target model's removed; the rotation is applied to the staged
 * tiles on chip (no extra pass over device memory).  The de-rotated rows are rounded to bf16 before they enter the
 * tensor cores.  Not available with CB_FLAG_SIMT (CB_ERR_UNSUPPORTED).
 *
 * cb_rope_rotate: stand-alone rotation of a strided bf16 key tensor IN PLACE (inverse != 0 removes the embedding),
 * element (layer, token, head, channel) at k + layer*stride_layer + token*stride_token + head*stride_head + channel,
 * alignment rules as for cb_kv_view.
 */
cb_status cb_stats_accumulate_rope(cb_ctx *ctx, const cb_kv_view *src, const cb_kv_view *tgt,
                                   const float *w_k, const float *w_v, int64_t w_stride_layer, int64_t w_stride_head,
                                   const int32_t *positions, double rope_base_src, double rope_base_tgt, void *stream);
cb_status cb_rope_rotate(void *k, int32_t n_layers, int32_t n_heads, int32_t head_dim, int64_t n_tokens,
                         int64_t stride_layer, int64_t stride_token, int64_t stride_head,
                         const int32_t *positions, double rope_base, int32_t inverse, void *stream);
/*
 * The two-pass centred construction (Section 3.4) with the rotary boundary (Section 3.1): both passes see the key rows
 * in content coordinates.  cb_means_accumulate_rope is cb_means_accumulate with the embedding removed from source and
 * target keys before they are summed (the means are those of the de-rotated rows, rounded to bf16 as the second pass
 * will see them); cb_stats_accumulate_centered_rope is cb_stats_accumulate_centered with the staged key tiles rotated
 * on chip as in cb_stats_accumulate_rope AND centred there (source and target), so that their rounding to bf16 is
 * relative to the spread of a channel, not to its mean.  Same call order as the plain two-pass path, same positions and
 * bases in both passes; between two resets either every chunk goes through the _rope call or none does (the context
 * remembers which, and cb_stats_reduce_centered skips the key maps' mean correction accordingly).  Both head widths.
 */
cb_status cb_means_accumulate_rope(cb_ctx *ctx, const cb_kv_view *src, const cb_kv_view *tgt,
                                   const float *w_k, const float *w_v, int64_t w_stride_layer, int64_t w_stride_head,
                                   void *means_ws, size_t means_ws_bytes,
                                   const int32_t *positions, double rope_base_src, double rope_base_tgt, void *stream);
cb_status cb_stats_accumulate_centered_rope(cb_ctx *ctx, const cb_kv_view *src, const cb_kv_view *tgt,
                                            const float *w_k, const float *w_v,
                                            int64_t w_stride_layer, int64_t w_stride_head, const float *mu,
                                            const int32_t *positions, double rope_base_src, double rope_base_tgt, void *stream);
/*
 * cb_apply_rope: as cb_apply, for a source cache whose keys carry the source model's rotary embedding and a target
 * cache that must carry the target model's:  K_out[l][t][h] = R_tgt(pos_t) ( R_src(-pos_t) x_t W + b ),  values as in
 * cb_apply.  Both rotations run inside the apply kernel (the staged source tile is rotated on chip, the mapped rows in
 * the epilogue).  The de-rotated keys enter the tensor cores as fp16 (11 significant bits; key magnitudes must stay
 * below 65504, the fp16 range, which bf16 caches of normalised keys do by orders of magnitude) with W split into fp16
 * hi + lo.  Not available with CB_FLAG_SIMT.
 */
cb_status cb_apply_rope(const cb_problem *prob, const float *Wb, const cb_kv_view *src_cache,
                        void *tgt_k, void *tgt_v, int64_t t_stride_layer, int64_t t_stride_token,
                        int64_t t_stride_head, int32_t out_dtype,
                        const int32_t *positions, double rope_base_src, double rope_base_tgt, void *stream);

/* ------------------------------------------------------------------------------------------------------------------
 * Layer selector (Section 3.1, first paragraph): for each target layer, centred single-source-layer least-squares
 * probes under the same head assignment, held-in R^2 averaged over KV heads and K/V, source layers ranked, the first k
 * taken.  Everything comes from statistics the path produces anyway:
 *   - a probe set = one cb_problem whose src_layer[] pairs every target layer with one candidate source layer; its
 *     statistics (cb_stats_accumulate .. cb_stats_reduce) and its fit (cb_ridge_solve with ONE lambda, 0 for the
 *     paper's OLS probe) are the ordinary ones; Ls probe sets with rotated src_layer[] cover every (l, j) pair;
 *   - the target's total sum of squares comes from the first pass of the two-pass path: cb_means_energy returns
 *     syy [n_maps][d] = sum w y^2 (device fp32) from a means workspace filled by cb_means_accumulate (the source side
 *     of that pass does not matter);
 *   - cb_probe_r2:  r2[m] = (tr(B^T W) + lambda_eff ||W||_F^2) / SST  with the centred B and SST formed from G, C, syy
 *     (= 1 - SSE/SST of the fitted probe, residuals pooled over the d channels: a reading, the paper does not say how
 *     channels are combined); G, C, Wb [n_maps][p][d] as produced for that lambda; r2 device fp32 [n_maps];
 *   - cb_probe_scores ADDS, for every target layer l, the mean of r2 over (K/V, head) to scores[l][src_layer[l]]
 *     (device fp32 [Lt][Ls], zeroed by the caller); src_layer is the HOST array of the probe set; Lt <= 128;
 *   - cb_rank_layers (host arrays): the k best source layers per target layer by descending score, ties to the lower
 *     index, written in ascending order as layer_sets [Lt][k] (the layout cb_fullhead_problem wants).
 */
cb_status cb_means_energy(cb_ctx *ctx, const void *means_ws, size_t means_ws_bytes, float *syy, void *stream);
cb_status cb_probe_r2(const float *G, const float *C, const float *Wb, const float *syy, int32_t n_maps, int32_t d,
                      int64_t n_tokens, float lambda, uint32_t flags, float *r2, void *stream);
cb_status cb_probe_scores(const float *r2, int32_t Lt, int32_t Ht, const int32_t *src_layer, int32_t Ls, float *scores,
                          void *stream);
cb_status cb_rank_layers(const float *scores, int32_t Lt, int32_t Ls, int32_t k, int32_t *layer_sets);

/*
 * Synchronises the stream and reads the context's device status word: CB_OK, or CB_ERR_TIMEOUT if a bounded
 * wait inside a kernel ran out (the statistics are then invalid; reset before reuse).
 */
cb_status cb_device_status(cb_ctx *ctx, void *stream);

/*
 * The same for the entry points that take no context (cb_apply, cb_apply_rope, cb_apply_multilayer,
 * cb_fullhead_stats_accumulate, cb_multilayer_stats_accumulate, cb_stats_build_static): their kernels record a
 * time-out in a status word that belongs to the library (one per device).  Synchronises the stream, returns
 * CB_ERR_TIMEOUT if any such kernel on the current device gave up since the last call (the outputs of that call are
 * then incomplete) and clears the word; CB_OK otherwise.  The paper has no counterpart: error reporting only.
 */
cb_status cb_last_device_status(void *stream);

/*
 * The CUDA runtime's error code behind the most recent CB_ERR_CUDA that any call of this library returned (0 if none
 * since the last call of this function), and, if `text` is not NULL, the runtime's description of it (a static
 * string owned by the runtime).  Reading clears it.  The paper has no counterpart: error reporting only.
 */
int32_t cb_last_cuda_error(const char **text);

/*
 * TEST HOOK, not for production use (the paper has no counterpart).  Affects every later launch of this process:
 * poll_limit > 0 shortens the number of polls after which a bounded device-side wait gives up (0 restores the
 * default of 2^22); starve_producer != 0 makes the source-tile producer of the statistics kernel (d = 128) and of
 * the apply kernel issue no copies at all, so that every consumer's bounded wait runs out, the blocks tear down by
 * themselves and the status word reads CB_ERR_TIMEOUT.  Nothing faults, traps or spins without a limit.
 */
cb_status cb_test_hooks(uint32_t poll_limit, int32_t starve_producer);

/*
 * Statistics of ONE batch of rows without any device allocation by anybody (the paper has no counterpart: this
 * entry point exists for deployment, not for the method).  It is for callers that cannot obtain scratch memory:
 * a serving process that gave all device memory to its own pool at start-up, an engine plug-in whose enqueue
 * hook must not call cudaMalloc (it synchronises the whole device), or a process running under a hard memory
 * cap.  Such callers cannot provide the workspace cb_create wants, so here the partial statistics live in a
 * fixed buffer of CB_STATIC_SCRATCH_MAX_BYTES that is part of the library image (every GPU that loads the
 * library holds it until the process exits).
 *
 * Computes the same G [n_maps][p][p] and C [n_maps][p][d] (device, fp32, caller-owned) that
 * cb_create + cb_stats_accumulate + cb_stats_reduce give for this one call's rows; arguments as for
 * cb_stats_accumulate, prob->n_splits == 0 means one split.  Work is enqueued on `stream`; the call itself
 * calls no cudaMalloc, cudaFree or other allocating routine.
 *   - Limit: n_splits * n_maps * (2 d^2 + 2 d + 4) * 4 bytes plus ~1 KB must fit in the buffer (e.g. 120 maps
 *     of d = 128 with one split); larger problems return CB_ERR_STATIC_LIMIT and nothing is enqueued.
 *   - The first call on each device looks up the buffer's device address (with that device current); make
 *     that first call outside any stream capture.  Every call also copies the two head tables of `prob` from
 *     host memory to the device on `stream`.
 *   - All calls on a device share the one buffer, which keeps the previous call's contents; each call clears
 *     what it needs on its stream first.  Two calls whose work overlaps on the GPU (different streams, no
 *     ordering between them) race on the buffer: order them.
 *   - There is no context: a device-side time-out shows in cb_last_device_status.
 */
#define CB_STATIC_SCRATCH_MAX_BYTES (16u << 20)
cb_status cb_stats_build_static(const cb_problem *prob, const cb_kv_view *src, const cb_kv_view *tgt,
                                const float *w_k, const float *w_v,
                                int64_t w_stride_layer, int64_t w_stride_head,
                                float *G, float *C, void *stream);

/* Number of kernels this library has launched in this process (all contexts); for accounting. */
int64_t cb_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* CB_H_ */
