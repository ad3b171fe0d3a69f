/*
 * astraea.h -- C ABI of the B200 (sm_100a) hot path of Astraea's per-denoising-step
 * token reduction for video diffusion transformers:
 *
 *     score -> select (budgeted top-k) -> sparse attention (selected queries x ALL
 *     keys/values) -> scatter over the cached output (unselected tokens reuse it).
 *
 * Conventions
 *   - Unless a parameter says "host", every data pointer is a DEVICE pointer owned by
 *     the caller.  The library never frees or retains caller memory and keeps no state
 *     between calls: all cross-step state (output cache, LSE cache, reference inputs,
 *     skip counters) lives in caller buffers.
 *   - Every call is asynchronous on `stream` (a cudaStream_t passed as void*; NULL is the
 *     default stream), does no host synchronisation and no device->host copy, except
 *     astraea_poll_error and astraea_step_host which say so.
 *   - Token order is [selectable tokens 0..N_sel) | always-kept tokens N_sel..N).
 *   - Hidden states and the cached attention output are [B, N, D] row-major bf16 with
 *     D = H*d and head h in columns [h*d, (h+1)*d), i.e. [B, N, H, d].
 *   - Return value: ASTRAEA_OK or a negative ASTRAEA_ERR_*.  Argument errors are found
 *     on the host before any launch and leave the outputs untouched;
 *     astraea_last_error() gives a text for the last failure on the calling thread.
 *   - Rows must start on 16-byte boundaries (d*2 and D*2 bytes are multiples of 16).
 *   - Inputs must not alias outputs except where "in place" is stated.
 */
#ifndef ASTRAEA_H
#define ASTRAEA_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define ASTRAEA_OK                        0
#define ASTRAEA_ERR_INVALID_ARG          -1  /* null/misaligned pointer, bad size, k outside [0,N_sel], D != H*d */
#define ASTRAEA_ERR_UNSUPPORTED          -2  /* head_dim not in {64,72,128}, unsupported flag or mode            */
#define ASTRAEA_ERR_WORKSPACE_TOO_SMALL  -3
#define ASTRAEA_ERR_CUDA                 -4  /* a CUDA call or launch failed                                      */
#define ASTRAEA_ERR_TIMEOUT              -5  /* a bounded device-side wait gave up (seen by astraea_poll_error)   */
#define ASTRAEA_ERR_BAD_INDEX            -6  /* an index list held an entry out of range or not strictly ascending
                                              * (found on the device; reported by astraea_poll_error)           */

#define ASTRAEA_N_SKIP_CLAMP 80              /* counters saturate here so that e^n stays finite in fp32 */
#define ASTRAEA_LSE_CLAMP    80              /* ASTRAEA_LSE_SUM_EXP: log values above this count as this, for the same reason */

/* delta_mode of astraea_score: how the per-token input difference is reduced over channels */
#define ASTRAEA_DELTA_MEAN_ABS    0          /* default reading: mean absolute difference */
#define ASTRAEA_DELTA_MEAN_SQ     1
#define ASTRAEA_DELTA_MEAN_SIGNED 2
/* lse_mode of astraea_score */
#define ASTRAEA_LSE_SUM_EXP 0                /* S_LSE = mean over heads of exp(lse): the paper's literal sum of exponentials */
#define ASTRAEA_LSE_LOG     1                /* S_LSE = mean over heads of lse itself */

/* flags of astraea_sparse_attn */
#define ASTRAEA_ATTN_COMPACT_OUT  1u         /* out is [B,M,H,d] and lse_out [B,H,M] (row r of the index list), not the caches */
#define ASTRAEA_ATTN_SMALL_CTAS   2u         /* head_dim 64 / 72: one 128-row query tile per CTA, two CTAs per SM, whatever the
                                              * launch-time estimate says (without the flag the library picks the faster shape) */
#define ASTRAEA_ATTN_WHOLE_KEYS   4u         /* every CTA runs over all keys: the last, partial round of CTAs is never split by keys
                                              * (see `workspace` of astraea_sparse_attn) */
/* flags of astraea_gathered_linear */
#define ASTRAEA_LINEAR_COMPACT_OUT 1u        /* y is [B,M,N_out] (row r of the index list), not the cache [B,N,N_out] */
#define ASTRAEA_LINEAR_COMPACT_IN  2u        /* x is [B,M,K]: row r is the row of token idx[b,r] (output of a layer run with COMPACT_OUT) */
#define ASTRAEA_LINEAR_GELU        4u        /* y = GELU(x W^T + bias), GELU(u) = u/2 (1 + erf(u / sqrt 2)): the first MLP layer
                                              * (erf in fp32 to 6e-7 absolute, before the one rounding to bf16) */
#define ASTRAEA_LINEAR_COMPACT_RES 8u        /* astraea_gathered_linear_residual: residual is [B,M,N_out] (row r of the index list) */
/* flags of astraea_layernorm_modulate */
#define ASTRAEA_LN_COMPACT_IN     1u         /* x is [B,M,D]: row r is the row of token idx[b,r] */
#define ASTRAEA_LN_COMPACT_OUT    2u         /* y is [B,M,D] */
/* flags of astraea_block_step */
#define ASTRAEA_BLOCK_REUSE_SELECTION 1u     /* idx_sel already holds this step's selection (made by another block): no scoring,
                                              * no selection, counters and reference inputs untouched (the Fixed-token variant) */
#define ASTRAEA_BLOCK_SELECT_QK   2u         /* keys and values of the self-attention are restricted to the selected tokens as well
                                              * (and projected for them only): the SelectQ&K variant of the ablation study, Table 2 */
/* variants of astraea_model_schedule_create: the rows of the ablation study (Table 2) */
#define ASTRAEA_VARIANT_TOKEN_WISE  0        /* the paper's method: every block scores and selects its own tokens at every step */
#define ASTRAEA_VARIANT_SELECT_QK   1        /* as above, with the self-attention also restricted to the selected keys / values */
#define ASTRAEA_VARIANT_TIMESTEP    2        /* Timestep-level: a step computes all tokens or none (budgets must be 0 or N_sel) */
#define ASTRAEA_VARIANT_FIXED_TOKEN 3        /* Fixed-token: block 0 selects, the other blocks of the step reuse its selection */
/* flags of astraea_scatter_reuse */
#define ASTRAEA_SCATTER_SRC_FULL  1u         /* rows is [B,N,row_elems]; row idx[r] of it is copied to row idx[r] of cache */

/* op codes of astraea_workspace_bytes */
#define ASTRAEA_OP_SELECT       1
#define ASTRAEA_OP_SPARSE_ATTN  2
#define ASTRAEA_OP_STEP         3
#define ASTRAEA_OP_SPARSE_ATTN_KV 4          /* astraea_sparse_attn with kv_idx: pass M_kv as the M argument */
#define ASTRAEA_OP_GATHERED_LINEAR 5        /* astraea_gathered_linear (the size arguments are ignored) */
#define ASTRAEA_OP_LAYERNORM    6            /* astraea_layernorm_modulate (the size arguments are ignored) */

/*
 * Selection metric (Section 3.2 "Selection Metric"; Algorithm 1 lines 1-2):
 *     S_token = w_alpha * S_LSE,t-1 * Delta_token,t + w_beta * e^{n_i}
 * for tokens [0, N_sel) of every batch row.  Delta_token is the difference between the
 * current inputs x_cur and the reference inputs x_ref (the inputs of the step at which
 * the token was last computed) reduced over the D channels as delta_mode says; S_LSE is
 * the softmax normaliser of the token's attention row from an earlier step, carried in
 * log domain and averaged over heads as lse_mode says; n_i counts the consecutive steps
 * in which token i was not selected (values above ASTRAEA_N_SKIP_CLAMP count as the clamp).
 * With ASTRAEA_LSE_SUM_EXP a log value above ASTRAEA_LSE_CLAMP counts as the clamp as well: e^lse of such a row
 * (one logit of 80 or more) would overflow fp32 and turn the scores of a whole batch row into inf / NaN.
 *   x_cur, x_ref : bf16 [B, N, D]                 lse    : fp32 [B, H, N]; NULL => S_LSE = 1
 *   n_skip       : int32 [B, N_sel]; NULL => 0    score  : out fp32 [B, N_sel]
 * Arithmetic: bf16 inputs, fp32 accumulation and result.
 * Errors: INVALID_ARG (null x/score, B,N,D,H <= 0, N_sel outside [0,N], D % 8 != 0,
 * pointers not 16-byte aligned), UNSUPPORTED (unknown mode), CUDA.
 */
int32_t astraea_score(const void *x_cur, const void *x_ref, const float *lse, const int32_t *n_skip,
                      float *score, int B, int N, int N_sel, int D, int H,
                      float w_alpha, float w_beta, int delta_mode, int lse_mode, void *stream);

/*
 * The selection metric when the heads (and with them the channels, D = H*d) are sharded over several GPUs (the
 * multi-GPU scalability experiment of Section 4; the paper does not name its scheme: here every GPU owns a
 * contiguous range of heads with the full-length keys / values, outputs and LSE values of those heads).  S_token is a
 * product of two sums that run over all channels and all heads, so each shard contributes raw partial sums,
 *     part[0, b, i] = sum over the shard's channels of |x_cur - x_ref| (or its square, or the signed difference)
 *     part[1, b, i] = sum over the shard's heads of exp(min(lse, ASTRAEA_LSE_CLAMP)) (or of lse in the log mode),
 * the partial sums of all shards are added up (ONE all-reduce of 2*B*N_sel floats), and astraea_score_combine turns
 * the totals into S_token = w_alpha * (part[1] / H) * (part[0] / D) + w_beta * e^n on every GPU alike, so that the
 * (deterministic) selection that follows is identical everywhere.
 *   x_cur, x_ref : bf16 [B, N, D_local]    lse : fp32 [B, H_local, N] or NULL (part[1] = 0)
 *   part         : out fp32 [2, B, N_sel]
 * astraea_score_combine: D, H are the TOTAL channel and head counts; has_lse = 0 => S_LSE = 1; n_skip may be NULL.
 * Errors: as astraea_score.
 */
int32_t astraea_score_partial(const void *x_cur, const void *x_ref, const float *lse, float *part,
                              int B, int N, int N_sel, int D_local, int H_local, int delta_mode, int lse_mode, void *stream);
int32_t astraea_score_combine(const float *part, const int32_t *n_skip, float *score, int B, int N_sel, int D, int H,
                              int has_lse, float w_alpha, float w_beta, void *stream);

/*
 * TopK(S_token, theta) -> I_sel, I_remain (Algorithm 1 line 3): the k largest scores of
 * each batch row.  Deterministic: equal scores go to the lower token index, -0 equals +0,
 * NaN ranks below every number.  Both index lists come out ascending by token index; the
 * always-kept span [N_sel, N_sel + n_always) is appended to idx_sel.  The skip counters
 * are updated in the same pass: 0 for a selected token, min(n+1, ASTRAEA_N_SKIP_CLAMP) otherwise.
 *   score   : fp32 [B, N_sel]
 *   idx_sel : out int32 [B, k + n_always]           idx_rem : out int32 [B, N_sel - k]; may be NULL
 *   n_skip  : in/out int32 [B, N_sel]; may be NULL
 *   workspace : at least astraea_workspace_bytes(ASTRAEA_OP_SELECT, B, 0, N_sel, k, 0) bytes, 16-byte aligned
 * k = 0 with n_always = 0 is valid (only the counters change).
 * Errors: INVALID_ARG (k outside [0,N_sel], negative sizes, null score/idx_sel when needed),
 * WORKSPACE_TOO_SMALL, CUDA.
 */
int32_t astraea_select(const float *score, int B, int N_sel, int k, int n_always,
                       int32_t *idx_sel, int32_t *idx_rem, int32_t *n_skip,
                       void *workspace, size_t workspace_bytes, void *stream);

/*
 * Sparse attention (Algorithm 1 line 6; Section 3.2 "Sparse Attention"; softmax and
 * attention equations of Section 3.1): for each listed query row i, head h,
 *     out[i] = Softmax(q_i K^T * scale) V   over ALL N keys/values,
 *     lse[i] = ln sum_j exp(q_i . k_j * scale),
 * written IN PLACE at row i of the caches (the reuse step of Algorithm 1 line 7 is thereby
 * fused: rows that are not listed keep their previous contents), or compactly with
 * ASTRAEA_ATTN_COMPACT_OUT.
 *   q, k, v : bf16, head_dim contiguous; element strides (batch, head, token) given per tensor.
 *             [B,N,H,d] has strides (N*H*d, d, H*d); [B,H,N,d] has (H*N*d, N*d, d).
 *             Token strides must be multiples of 8 elements, bases 16-byte aligned.
 *   q_idx   : int32 [B, M] strictly ascending token indices in [0,N); NULL => rows 0..M-1.  An entry out of
 *             range, or one that does not exceed its predecessor (a duplicate, a descending step), is never
 *             dereferenced or written: its row is skipped and astraea_poll_error reports BAD_INDEX.
 *   kv_idx  : NULL (all keys: the paper's method), or int32 [B, M_kv] token indices in [0,N): the softmax then
 *             runs over the listed keys/values only (the SelectQ&K variant of the paper's ablation study, Table 2).  Their
 *             rows are gathered into the workspace first, which must then hold
 *             astraea_workspace_bytes(ASTRAEA_OP_SPARSE_ATTN_KV, B, H, N, M_kv, d) bytes.
 *   out     : bf16 [B, N, H, d]  (or [B, M, H, d] compact)
 *   lse_out : fp32 [B, H, N]     (or [B, H, M] compact); may be NULL
 *   scale   : 0 => 1/sqrt(d)
 *   workspace : 256-byte aligned, at least 256 bytes (with kv_idx: see above); its first word is an error word (see
 *               astraea_poll_error).  With astraea_workspace_bytes(ASTRAEA_OP_SPARSE_ATTN, B, H, N, M, d) bytes (a few
 *               tens of MB at most) a launch of only a few rounds of CTAs may split the keys of its last, partial round:
 *               each of those CTAs is replaced by 2..8 CTAs that take a share of the keys each and leave fp32 rows
 *               in the workspace, which a second kernel merges (out = sum_i exp(lse_i - lse) out_i).  Results agree
 *               with the unsplit launch to fp32 rounding.  A workspace serves one call at a time.
 * Arithmetic: bf16 operands, fp32 logits, softmax and accumulation; probabilities are
 * rounded to bf16 before the P.V product; outputs rounded to bf16.
 * M = 0 is valid: nothing is launched and the caches are untouched.
 * Errors: INVALID_ARG, UNSUPPORTED (d not in {64,72,128}), WORKSPACE_TOO_SMALL, CUDA.
 */
int32_t astraea_sparse_attn(const void *q, const void *k, const void *v,
                            int64_t q_sb, int64_t q_sh, int64_t q_sn,
                            int64_t k_sb, int64_t k_sh, int64_t k_sn,
                            int64_t v_sb, int64_t v_sh, int64_t v_sn,
                            const int32_t *q_idx, int M, const int32_t *kv_idx, int M_kv,
                            void *out, float *lse_out,
                            int B, int H, int N, int d, float scale, uint32_t flags,
                            void *workspace, size_t workspace_bytes, void *stream);

/*
 * The launch schedule astraea_sparse_attn would pick for a problem (host logic only, no GPU work): small_ctas = 1 when
 * it launches one query tile per CTA; otherwise the last split_units CTAs are replaced by `split` CTAs each that share
 * the keys (split = 1, split_units = 0: every CTA runs over all keys).  workspace_bytes as given to astraea_sparse_attn.
 * Errors: INVALID_ARG, UNSUPPORTED.
 */
int32_t astraea_sparse_attn_plan(int B, int H, int N, int M, int d, uint32_t flags, size_t workspace_bytes,
                                 int32_t *small_ctas, int32_t *split_units, int32_t *split);

/*
 * Cross-attention of the selected rows (Section 3.2: the layers of a block other than self-attention are
 * computed for the selected tokens only and their cached results reused for the rest): as
 * astraea_sparse_attn, but keys and values come from another sequence of N_kv tokens (the text tokens),
 *     out[b, i, h, :] = Softmax(q[b, i, h, :] K[b, :, h, :]^T * scale) V[b, :, h, :]   for i in q_idx,
 * k, v : bf16 [B, N_kv, H, d] through their stride triples; q, out, lse_out, q_idx, M, flags, workspace as above
 *        (the keys that a launch may split are the N_kv ones: size the workspace with N_kv in place of N for that)
 * (N is the token count of q and out).  There is no kv_idx form.  Errors as astraea_sparse_attn.
 */
int32_t astraea_sparse_cross_attn(const void *q, const void *k, const void *v,
                                  int64_t q_sb, int64_t q_sh, int64_t q_sn,
                                  int64_t k_sb, int64_t k_sh, int64_t k_sn,
                                  int64_t v_sb, int64_t v_sh, int64_t v_sn,
                                  const int32_t *q_idx, int M, void *out, float *lse_out,
                                  int B, int H, int N, int N_kv, int d, float scale, uint32_t flags,
                                  void *workspace, size_t workspace_bytes, void *stream);

/*
 * The same attention for callers that must not allocate.  (The paper has no counterpart: this is a
 * property of the library, not of the method.)  astraea_sparse_attn takes its scratch from the
 * caller, which some callers cannot provide: code that runs while a CUDA memory pool or a framework
 * allocator is locked, inside a region where cudaMalloc would synchronise the device, or in a
 * process whose device memory has been handed out in full to other owners.  This entry point keeps
 * its scratch in a fixed array inside the library image instead (ASTRAEA_NOALLOC_SCRATCH_BYTES per
 * GPU that loads the library, held until the process exits) and calls no cudaMalloc, cudaFree or
 * other allocating routine.  Arguments (flags included), validation, arithmetic and results are those of
 * astraea_sparse_attn without the workspace pair: the two entry points share one code path.
 *   - Without kv_idx the 256 bytes every launch needs fit the array: nothing is rejected for its size, and
 *     the launch never splits its last round of CTAs by keys (there is no room for the shares).  With kv_idx a problem
 *     whose need (astraea_workspace_bytes(ASTRAEA_OP_SPARSE_ATTN_KV, ...)) exceeds ASTRAEA_NOALLOC_SCRATCH_BYTES is
 *     rejected with ASTRAEA_ERR_WORKSPACE_TOO_SMALL, which is nearly always the case: the gathered key / value
 *     rows (2 * B * M_kv * H * d bf16) must fit the array.
 *   - The first call on a device resolves the array's device address (with that device current);
 *     make that first call before any stream capture.
 *   - All calls on a device share the one array.  It keeps the last call's contents, so each call
 *     first clears its error word on `stream` (also a call that is then rejected for its arguments); calls
 *     that overlap on the GPU (different streams) race on it and must be serialised by the caller.
 *   - The error word lives in that array, so astraea_poll_error cannot be pointed at it: a device-side
 *     timeout or bad index in this variant is not reported.  Callers that need the report use
 *     astraea_sparse_attn.
 * Errors: INVALID_ARG, UNSUPPORTED, WORKSPACE_TOO_SMALL (see above), CUDA.
 */
#define ASTRAEA_NOALLOC_SCRATCH_BYTES 4096
int32_t astraea_sparse_attn_noalloc(const void *q, const void *k, const void *v,
                                    int64_t q_sb, int64_t q_sh, int64_t q_sn,
                                    int64_t k_sb, int64_t k_sh, int64_t k_sn,
                                    int64_t v_sb, int64_t v_sh, int64_t v_sn,
                                    const int32_t *q_idx, int M, const int32_t *kv_idx, int M_kv,
                                    void *out, float *lse_out,
                                    int B, int H, int N, int d, float scale, uint32_t flags, void *stream);

/*
 * Reuse / cache update (Algorithm 1 lines 6-7; Section 3.2 "Execution Flow"):
 *     cache[b, idx[b,r], :] = rows[b, r, :]      (rows compact [B, M, row_elems]), or
 *     cache[b, idx[b,r], :] = rows[b, idx[b,r], :] with ASTRAEA_SCATTER_SRC_FULL;
 * every row that is not listed is left untouched, i.e. keeps the earlier step's value.
 * The second form refreshes the reference inputs of the tokens that were computed.
 *   cache : bf16 [B, N, row_elems], in place      rows : bf16
 *   idx   : int32 [B, M], strictly ascending in [0,N).  An entry out of range or not above its predecessor is
 *           skipped (nothing is written outside the cache, no row is written twice).
 *   err_workspace : NULL, or any workspace of this library (at least 4 bytes, 4-byte aligned): its first word is
 *           the error word, and a skipped entry is then reported as BAD_INDEX by astraea_poll_error.  With NULL
 *           such entries are skipped without a report.
 * M = 0 is valid.  Errors: INVALID_ARG (row_elems % 8 != 0, misaligned pointers, ...), CUDA.
 */
int32_t astraea_scatter_reuse(void *cache, const void *rows, const int32_t *idx,
                              int B, int N, int M, int row_elems, uint32_t flags,
                              void *err_workspace, void *stream);

/*
 * A linear layer of the compute block on the selected tokens only (Algorithm 1 lines 4-5: the query
 * projection X_in[I_sel] W_Q of the gathered rows, the key / value projections of all rows; Section 3.2:
 * the other layers of the block follow the same gather - compute - scatter pattern):
 *     y[b, idx[b,r], :] = x[b, idx[b,r], :] W^T + bias        for r in [0, M)
 * and every row of y that is not listed is left untouched, i.e. keeps the cached result of the earlier
 * step.  The gather of the rows of x and the scatter of the rows of y are fused into the GEMM.
 *   x    : bf16 [B, N, K] (with ASTRAEA_LINEAR_COMPACT_IN bf16 [B, M, K])
 *   idx  : int32 [B, M] strictly ascending in [0,N); NULL => all N rows (M ignored)
 *   w    : bf16 [N_out, K] row-major (out features x in features)        bias : bf16 [N_out] or NULL
 *   y    : bf16 [B, N, N_out], rows at idx written in place; with ASTRAEA_LINEAR_COMPACT_OUT bf16 [B, M, N_out]
 *   workspace : at least astraea_workspace_bytes(ASTRAEA_OP_GATHERED_LINEAR, 0, 0, 0, 0, 0) bytes, 256-byte
 *               aligned, zero before the first use (holds the error word read by astraea_poll_error).
 * With ASTRAEA_LINEAR_COMPACT_OUT on the first and ASTRAEA_LINEAR_COMPACT_IN on the second layer the hidden
 * activations of the MLP exist for the selected rows only.
 * bf16 operands, fp32 accumulation (and fp32 GELU), one rounding to bf16 at the end.  K must be a multiple of 64, N_out
 * a multiple of 8; x, w, y 16-byte aligned.  M = 0 is valid (nothing is launched).  An index outside
 * [0,N), or one that does not exceed its predecessor, is not dereferenced: its row is skipped and
 * astraea_poll_error reports BAD_INDEX.
 * Errors: INVALID_ARG, UNSUPPORTED (unknown flags), WORKSPACE_TOO_SMALL, CUDA.
 */
int32_t astraea_gathered_linear(const void *x, const int32_t *idx, int M, const void *w, const void *bias,
                                void *y, int B, int N, int K, int N_out, uint32_t flags,
                                void *workspace, size_t workspace_bytes, void *stream);

/*
 * The same layer with a gated residual in its epilogue (the residual connections around the layer groups of a
 * compute block, applied to the selected rows only, Section 3.2):
 *     y[b, idx[b,r], :] = residual[b, idx[b,r], :] + gate[b, :] * act(x[b, idx[b,r], :] W^T + bias)
 *   residual : bf16 [B, N, N_out] (rows at idx), with ASTRAEA_LINEAR_COMPACT_RES bf16 [B, M, N_out]; NULL => none
 *   gate     : bf16 [B, N_out] or NULL (no gate)
 * Everything else as astraea_gathered_linear; fp32 until the one rounding to bf16 at the end.
 */
int32_t astraea_gathered_linear_residual(const void *x, const int32_t *idx, int M, const void *w, const void *bias,
                                         const void *residual, const void *gate,
                                         void *y, int B, int N, int K, int N_out, uint32_t flags,
                                         void *workspace, size_t workspace_bytes, void *stream);

/*
 * Layer normalisation and modulation of token rows, the element-wise step in front of the layer groups of a compute
 * block (Section 3.2: the layers other than self-attention act on each token by itself, so it runs for the selected
 * rows only; in front of the key / value projections, Algorithm 1 line 4, for all rows):
 *     y[b, idx[b,r], :] = (x[b, idx[b,r], :] - mean) / sqrt(var + eps) * (1 + scale[b, :]) + shift[b, :]
 * with mean and the biased variance over the D channels of the row and no learned affine.
 *   x : bf16 [B, N, D] (ASTRAEA_LN_COMPACT_IN: [B, M, D])     y : bf16 [B, N, D] (ASTRAEA_LN_COMPACT_OUT: [B, M, D])
 *   idx : int32 [B, M] strictly ascending in [0,N); NULL => all N rows (M ignored, compact flags not allowed)
 *   scale, shift : bf16 [B, D] or NULL
 *   err_workspace : NULL, or any workspace of this library: bad index entries are skipped and then reported there
 * fp32 arithmetic, one rounding to bf16.  D a multiple of 8, at most 4096; pointers 16-byte aligned.
 * Errors: INVALID_ARG, UNSUPPORTED (D too large, unknown flags), CUDA.
 */
int32_t astraea_layernorm_modulate(const void *x, const int32_t *idx, int M, const void *scale, const void *shift,
                                   void *y, int B, int N, int D, float eps, uint32_t flags,
                                   void *err_workspace, void *stream);

/*
 * One whole compute block (self-attention, cross-attention, MLP; pre-norm, residual) at one denoising step with
 * token-wise reuse: Algorithm 1 and the execution flow of Section 3.2 applied to every layer of the block.  The
 * tokens are scored on the block's input x and selected (as astraea_step does); keys and values are projected from
 * ALL tokens of the current step (Algorithm 1 line 4); the query projection (line 5), the self-attention rows (line
 * 6), the output projection, the cross-attention against the text keys / values and the MLP run for the selected
 * rows only, on compact buffers; the block's cached output keeps every other row (line 7).  With I = idx_sel:
 *     h        = LN(x) (1 + s1) + t1                        all rows
 *     K, V     = h Wk^T + bk, h Wv^T + bv                   all rows;      Q[I] = h[I] Wq^T + bq
 *     x1       = x[I] + g1 * (Attn(Q[I], K, V) Wo^T + bo)
 *     x2       = x1 + Attn(LN(x1) Wq2^T + bq2, text_k, text_v) Wo2^T + bo2
 *     y_cache[I] = x2 + g3 * (GELU((LN(x2) (1 + s3) + t3) W1^T + b1) W2^T + b2)
 *     lse_cache[:, I] = LSE of the self-attention rows;  x_ref[I] = x[I];  counters as astraea_select
 * All tensors bf16 device memory; weights [out features, in features] row-major; biases [out]; modulation vectors
 * [B, D]; any bias or modulation pointer may be NULL.  text_k, text_v: [B, N_text, H, d] (projected once per
 * generation by the caller).  State (in/out): x_ref [B,N,D], lse_cache fp32 [B,H,N], n_skip int32 [B,N_sel], y_cache
 * [B,N,D] = the block's output after the call.  score / idx_sel / idx_rem as astraea_step.
 * flags: ASTRAEA_BLOCK_REUSE_SELECTION, ASTRAEA_BLOCK_SELECT_QK (see there).
 * workspace: astraea_block_workspace_bytes(B, H, N, d, hidden) bytes, 256-byte aligned, zero before the first use.
 * D = H*d must be a multiple of 64 and at most 4096, hidden a multiple of 64.
 * k_keep = 0 with no always-kept tokens: only scores and counters change.
 * Errors: as the calls it is made of.
 */
typedef struct astraea_block_weights {
    const void *wq, *bq, *wk, *bk, *wv, *bv, *wo, *bo;      /* self-attention: D x D each */
    const void *wq2, *bq2, *wo2, *bo2;                      /* cross-attention query / output projection: D x D */
    const void *w1, *b1, *w2, *b2;                          /* MLP: hidden x D, D x hidden */
    const void *s1, *t1, *g1, *s3, *t3, *g3;                /* scale, shift, gate of the attention and MLP groups: [B, D] */
    int32_t hidden;
} astraea_block_weights;
typedef struct astraea_block_state {
    void *x_ref; float *lse_cache; int32_t *n_skip; void *y_cache;
} astraea_block_state;
size_t  astraea_block_workspace_bytes(int B, int H, int N, int d, int hidden);
int32_t astraea_block_step(const void *x, const astraea_block_weights *weights, const astraea_block_state *state,
                           const void *text_k, const void *text_v, int N_text,
                           float *score, int32_t *idx_sel, int32_t *idx_rem,
                           int B, int H, int N, int N_sel, int d, int k_keep,
                           float w_alpha, float w_beta, int delta_mode, int lse_mode, float eps, uint32_t flags,
                           void *workspace, size_t workspace_bytes, void *stream);

/*
 * A generation as ONE CUDA graph: T denoising steps x L compute blocks (the execution flow of Section 3.2 with the
 * per-step budgets theta_t of the search space of Section 3.3, fixed before the generation starts).  At step t block
 * 0 reads x_in[t]; block l > 0 reads block l-1's merged output of the same step (its y_cache: computed rows + reused
 * rows); every block keeps its own state (reference inputs, LSE cache, counters, output cache) and, per block,
 * score / idx_sel / idx_rem buffers that hold its last selection.  `variant` picks the row of the ablation study
 * (Table 2): the paper's token-wise method, SelectQ&K, Timestep-level (every budget 0 or N_sel: the policy
 * astraea_timestep_level_budgets makes such a schedule from a token-wise one) or Fixed-token (block 0's selection is
 * shared by all blocks of the step; the other blocks' counters and reference inputs are not used).
 *   k_keep : HOST int32 [T]                     x_in : HOST array of T device pointers, bf16 [B,N,D] each
 *   weights, states : HOST arrays of L structs  text_k, text_v : HOST arrays of L device pointers, bf16 [B,N_text,H,d]
 *   score, idx_sel, idx_rem : HOST arrays of L device pointers (fp32 [B,N_sel]; int32 [B,N]; int32 [B,N_sel] or NULL)
 *   workspace : astraea_block_workspace_bytes(...) bytes, shared by all blocks (they run one after the other)
 * The first step of a generation should carry k_keep = N_sel.  The graph keeps the pointers, not the data.
 * astraea_model_schedule_launch enqueues the whole generation with one graph launch; the last block's y_cache then
 * holds the output of the last step.  Errors: as astraea_block_step, INVALID_ARG for a budget the variant does not
 * allow, CUDA for a failed capture.
 */
typedef struct astraea_model_schedule astraea_model_schedule;
int32_t astraea_model_schedule_create(astraea_model_schedule **schedule, int L, int T, const int32_t *k_keep,
                                      const void *const *x_in, const astraea_block_weights *weights,
                                      const astraea_block_state *states, const void *const *text_k,
                                      const void *const *text_v, int N_text,
                                      float *const *score, int32_t *const *idx_sel, int32_t *const *idx_rem,
                                      int B, int H, int N, int N_sel, int d,
                                      float w_alpha, float w_beta, int delta_mode, int lse_mode, float eps, int variant,
                                      void *workspace, size_t workspace_bytes);
int32_t astraea_model_schedule_launch(astraea_model_schedule *schedule, void *stream);
void    astraea_model_schedule_destroy(astraea_model_schedule *schedule);

/*
 * Host policy of the Timestep-level variant (ablation study, Table 2): turns a token-wise budget schedule into one
 * whose steps compute all tokens or none, with the same total budget up to one step: the budgets are accumulated and
 * a step computes everything as soon as the accumulated budget covers N_sel tokens (the first step always does).
 *   k_keep, out : HOST int32 [T] (may be the same array).  Returns the number of computed steps, or INVALID_ARG.
 */
int32_t astraea_timestep_level_budgets(const int32_t *k_keep, int T, int N_sel, int32_t *out);

/*
 * One whole step of one attention block on device buffers (Algorithm 1 with given Q, K, V):
 * score -> select -> sparse attention with fused scatter -> refresh of x_ref at the
 * selected tokens.  Equivalent to the four calls above in sequence on `stream`.
 *   x_cur : bf16 [B,N,D]       x_ref : in/out bf16 [B,N,D]   lse_cache : in/out fp32 [B,H,N]
 *   n_skip: in/out int32 [B,N_sel]                           q,k,v     : bf16 [B,N,H,d]
 *   out_cache : in/out bf16 [B,N,H,d]
 *   score : scratch/out fp32 [B,N_sel]   idx_sel : out int32 [B,k+n_always]   idx_rem : out int32 [B,N_sel-k] or NULL
 *   workspace : astraea_workspace_bytes(ASTRAEA_OP_STEP, B, H, N, k + n_always, d) bytes
 */
int32_t astraea_step(const void *x_cur, void *x_ref, float *lse_cache, int32_t *n_skip,
                     const void *q, const void *k, const void *v, void *out_cache,
                     float *score, int32_t *idx_sel, int32_t *idx_rem,
                     int B, int H, int N, int N_sel, int d, int k_keep,
                     float w_alpha, float w_beta, int delta_mode, int lse_mode,
                     void *workspace, size_t workspace_bytes, void *stream);

/*
 * A schedule of T denoising steps of one attention block as ONE CUDA graph (the per-step token budgets
 * theta_t of Section 3.3 are fixed before the generation starts, so the whole loop of Algorithm 1 can be
 * recorded once and replayed): step t runs astraea_step with budget k_keep[t] on the inputs x_cur[t], q[t],
 * k[t], v[t] and the shared state.  A budget of 0 with no always-kept tokens skips the attention of that step
 * (scores and counters are still updated); the first step of a generation should carry k_keep = N_sel.
 * astraea_schedule_create captures and instantiates the graph (host work only, nothing runs on the device);
 * astraea_schedule_launch enqueues all T steps on `stream` with a single graph launch, asynchronously.
 *   k_keep            : HOST int32 [T]
 *   x_cur, q, k, v    : HOST arrays of T DEVICE pointers (bf16 [B,N,D] each; the producers of those tensors,
 *                       i.e. the rest of the model, are outside this library)
 *   x_ref ... idx_rem, workspace : device buffers as for astraea_step; idx_sel holds at least B*N entries,
 *                       idx_rem at least B*N_sel (or NULL), workspace the ASTRAEA_OP_STEP size for M = N
 * The graph keeps the pointers, not the data: the buffers must stay allocated while the schedule exists and
 * may be refilled between launches.  Errors: as astraea_step, plus CUDA for a failed capture.
 */
typedef struct astraea_schedule astraea_schedule;
int32_t astraea_schedule_create(astraea_schedule **schedule, int T, const int32_t *k_keep,
                                const void *const *x_cur, const void *const *q, const void *const *k,
                                const void *const *v, void *x_ref, float *lse_cache, int32_t *n_skip,
                                void *out_cache, float *score, int32_t *idx_sel, int32_t *idx_rem,
                                int B, int H, int N, int N_sel, int d,
                                float w_alpha, float w_beta, int delta_mode, int lse_mode,
                                void *workspace, size_t workspace_bytes);
int32_t astraea_schedule_launch(astraea_schedule *schedule, void *stream);
void    astraea_schedule_destroy(astraea_schedule *schedule);

/*
 * Host-buffer session: the library owns the device-side state of one attention block
 * (x_ref, LSE cache, counters, output cache) and staging buffers, and each step copies
 * the HOST inputs to the device, runs the step (score, select, refresh of x_ref,
 * sparse attention) and copies the merged output back.  The copies run on streams of
 * their own: x_cur goes first, q / k / v follow in up to twelve groups of heads, the attention
 * of a group starts when its heads have arrived, and the group's columns of the output
 * go back while the next group is computed.  The results are those of astraea_step.
 * astraea_session_create allocates device memory (cudaMalloc) on the current device;
 * the first step of a session must be run with k_keep = N_sel (all tokens computed) to
 * fill the caches, as the paper's denoising loop does at its first timestep.
 *   x_cur, q, k, v : host bf16 [B,N,D] (pinned memory gives asynchronous copies; from a pinned q only the rows of
 *                    the selected tokens cross the bus: the rest of q is never read)
 *   out            : host bf16 [B,N,D], receives X_out,t (computed + cached rows)
 * astraea_step_host synchronises the session's streams before it returns.
 */
typedef struct astraea_session astraea_session;
int32_t astraea_session_create(astraea_session **session, int B, int H, int N, int N_sel, int d);
void    astraea_session_destroy(astraea_session *session);
int32_t astraea_step_host(astraea_session *session, const void *x_cur, const void *q, const void *k,
                          const void *v, void *out, int k_keep,
                          float w_alpha, float w_beta, int delta_mode, int lse_mode);
/* Host-to-device bytes that the last astraea_step_host of the session moved (0 before the first step). */
size_t  astraea_session_last_h2d_bytes(const astraea_session *session);

/* Scratch size for an op (bytes); 0 for unknown ops.  H, d, M may be 0 where the op does not use them. */
size_t  astraea_workspace_bytes(int op, int B, int H, int N, int M, int d);

/* k = floor(n_sel * theta_permille / 1000) in integer arithmetic (budget theta in 1/1000). */
int32_t astraea_budget_to_k(int n_sel, int theta_permille);

/*
 * Synchronises `stream`, reads the error word at the start of `workspace` and clears it.
 * Returns ASTRAEA_OK, ASTRAEA_ERR_TIMEOUT, ASTRAEA_ERR_BAD_INDEX or ASTRAEA_ERR_CUDA.
 */
int32_t astraea_poll_error(void *workspace, void *stream);

/*
 * Self-test of the failure detection: every wait inside the tensor-core kernels (on a copy, an MMA, another warp) is
 * bounded; when one runs out the kernel raises ASTRAEA_ERR_TIMEOUT in its workspace's error word, lets its remaining
 * waits return at once and exits in order.  This call runs that give-up path in isolation: one warp waits for at most
 * limit_us microseconds (1 .. 1000) on a barrier that nothing ever arrives at, then returns.  Afterwards
 * astraea_poll_error(workspace) reports ASTRAEA_ERR_TIMEOUT and the context and the workspace remain usable.
 *   gave_up : optional device int32, set to 1 by the kernel when its wait ran out
 * (The paper has no counterpart: this is a property of the library.)
 */
int32_t astraea_selftest_wait(void *workspace, int limit_us, int32_t *gave_up, void *stream);

const char *astraea_last_error(void);
const char *astraea_version(void);

#ifdef __cplusplus
}
#endif
#endif /* ASTRAEA_H */
