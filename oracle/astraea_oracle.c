/*
 * CPU oracle for Astraea's per-step token reduction (score -> select -> sparse
 * attention -> reuse).  TEST INFRASTRUCTURE ONLY: it exists to check the CUDA
 * library and to be timed as a CPU baseline.  It shares no code, header, table
 * or constant with the CUDA path, and the product never calls it.
 *
 * Everything is the plain definition, in fp64, in the paper's order:
 *   - no blocking, no online softmax, no fused steps;
 *   - OpenMP only over independent outer iterations (tokens / query rows).
 *
 * Readings taken where the paper is silent or inconsistent are marked [Rn] and
 * listed in the repository's design notes:
 *   [R1] Delta_token is the mean ABSOLUTE difference over channels (modes for the
 *        squared and the signed mean exist as well).
 *   [R3] the "LSE score" is carried as ln(sum exp) and turned back into the sum
 *        of exponentials at scoring time (mode 1 uses the log value itself).  The
 *        paper's sum of exponentials has no bound, fp32 has: a log value above 80
 *        counts as 80 (as for n_i in [R8]), so that the fp32 scores stay finite.
 *   [R4] per-head LSE scores are averaged over heads.
 *   [R8] n_i is reset to 0 when token i is selected, incremented otherwise, and
 *        clamped to 80 so that e^{n_i} stays finite in fp32.
 *   [R10] ties go to the lower token index; NaN scores rank below everything.
 *   [R11] index lists are ascending by token index.
 *   [R12] tokens [N_sel, N_sel + n_always) are never scored and always selected.
 *
 * Parity pins (tests/test_oracle_pins.py): dense special case vs an independent
 * library softmax-attention; keep-ratio 0 identity; brute-force selection;
 * softmax rows sum to 1; closed forms for zero keys, constant values, a dominant
 * key, constant per-token differences, the round-robin penalty schedule;
 * permutation invariances; half-normal drift statistics; the linear layer on listed rows
 * vs a library matmul, a one-hot weight, a zero weight and pure-Python brute force; the
 * LSE scatter vs numpy indexing; a whole step at a partial budget (computed rows vs the
 * dense library attention, cached rows / LSE / reference inputs untouched elsewhere).
 * parity unpinned: absolute score values under the paper's own (unpublished)
 * w_alpha, w_beta and its intended reading of [R1]-[R4].
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_N_CLAMP 80
#define ORACLE_LSE_CLAMP 80.0

/* ------------------------------------------------------------------ score
 * Selection metric, Eq. for S_token = w_a * S_sig + w_b * S_penalty with
 * S_sig = S_LSE,t-1 * Delta_token,t and S_penalty = e^{n_i} (Section 3.2,
 * "Selection Metric"; Algorithm 1 lines 1-2).
 *   x_cur, x_ref : [B, N, D]   lse : [B, H, N] (log domain) or NULL (S_LSE = 1)
 *   n_skip       : [B, N_sel] or NULL (all zero)    score : [B, N_sel]
 *   delta_mode 0: mean |.|   1: mean (.)^2   2: signed mean
 *   lse_mode   0: S_LSE = mean_h exp(lse)    1: S_LSE = mean_h lse
 */
void oracle_score(const double *x_cur, const double *x_ref, const double *lse,
                  const int32_t *n_skip, double *score,
                  int B, int N, int N_sel, int D, int H,
                  double w_alpha, double w_beta, int delta_mode, int lse_mode)
{
    for (int b = 0; b < B; ++b) {
#pragma omp parallel for schedule(static)
        for (int i = 0; i < N_sel; ++i) {
            const double *xc = x_cur + ((size_t)b * N + i) * D;
            const double *xr = x_ref + ((size_t)b * N + i) * D;
            double acc = 0.0;
            for (int c = 0; c < D; ++c) {
                double diff = xc[c] - xr[c];
                if (delta_mode == 0) acc += fabs(diff);
                else if (delta_mode == 1) acc += diff * diff;
                else acc += diff;
            }
            double delta = acc / (double)D;
            double s_lse = 1.0;
            if (lse) {
                double a = 0.0;
                for (int h = 0; h < H; ++h) {
                    double l = lse[((size_t)b * H + h) * N + i];
                    if (lse_mode == 0 && l > ORACLE_LSE_CLAMP) l = ORACLE_LSE_CLAMP;      /* [R3] */
                    a += (lse_mode == 0) ? exp(l) : l;
                }
                s_lse = a / (double)H;
            }
            int n = n_skip ? n_skip[(size_t)b * N_sel + i] : 0;
            if (n > ORACLE_N_CLAMP) n = ORACLE_N_CLAMP;
            double s_sig = s_lse * delta;
            double s_pen = exp((double)n);
            score[(size_t)b * N_sel + i] = w_alpha * s_sig + w_beta * s_pen;
        }
    }
}

/* ----------------------------------------------------------------- select
 * TopK(S_token, theta) -> I_sel, I_remain (Algorithm 1 line 3).  The whole
 * score row is sorted with a stable merge sort by descending score, so equal
 * scores stay in ascending index order; the first k entries are the selection.
 * Scores are compared as the fp32 values they are given in.
 *   idx_sel : [B, k + n_always] ascending, the always-kept span appended
 *   idx_rem : [B, N_sel - k] ascending (may be NULL)
 *   n_skip  : [B, N_sel] in/out (may be NULL)
 * Returns 0, or -1 for a bad k.
 */
static float rank_value(float s) { return isnan(s) ? -INFINITY : s; }

static void stable_sort_desc(const float *key, int32_t *idx, int32_t *tmp, int n)
{
    for (int width = 1; width < n; width *= 2) {
        for (int lo = 0; lo < n; lo += 2 * width) {
            int mid = lo + width < n ? lo + width : n;
            int hi = lo + 2 * width < n ? lo + 2 * width : n;
            int a = lo, c = mid, o = lo;
            while (a < mid && c < hi) {
                /* take from the right run only when it is strictly larger */
                if (rank_value(key[idx[c]]) > rank_value(key[idx[a]])) tmp[o++] = idx[c++];
                else tmp[o++] = idx[a++];
            }
            while (a < mid) tmp[o++] = idx[a++];
            while (c < hi) tmp[o++] = idx[c++];
        }
        memcpy(idx, tmp, (size_t)n * sizeof(int32_t));
    }
}

int oracle_select(const float *score, int B, int N_sel, int k, int n_always,
                  int32_t *idx_sel, int32_t *idx_rem, int32_t *n_skip)
{
    if (k < 0 || k > N_sel || n_always < 0) return -1;
    int32_t *order = (int32_t *)malloc((size_t)(N_sel + 1) * sizeof(int32_t));
    int32_t *tmp = (int32_t *)malloc((size_t)(N_sel + 1) * sizeof(int32_t));
    uint8_t *chosen = (uint8_t *)malloc((size_t)N_sel + 1);
    for (int b = 0; b < B; ++b) {
        const float *s = score + (size_t)b * N_sel;
        for (int i = 0; i < N_sel; ++i) order[i] = i;
        stable_sort_desc(s, order, tmp, N_sel);
        memset(chosen, 0, (size_t)N_sel + 1);
        for (int r = 0; r < k; ++r) chosen[order[r]] = 1;
        int ns = 0, nr = 0;
        int32_t *sel = idx_sel + (size_t)b * (k + n_always);
        int32_t *rem = idx_rem ? idx_rem + (size_t)b * (N_sel - k) : NULL;
        for (int i = 0; i < N_sel; ++i) {
            if (chosen[i]) sel[ns++] = i;
            else if (rem) rem[nr++] = i;
            if (n_skip) {
                int32_t *n = n_skip + (size_t)b * N_sel + i;
                if (chosen[i]) *n = 0;
                else *n = (*n + 1 > ORACLE_N_CLAMP) ? ORACLE_N_CLAMP : *n + 1;
            }
        }
        for (int t = 0; t < n_always; ++t) sel[ns++] = N_sel + t;
    }
    free(order); free(tmp); free(chosen);
    return 0;
}

/* ------------------------------------------------------------ sparse attn
 * X_out[I_sel] = Softmax(Q_sel K^T / sqrt(d)) V with ALL keys and values
 * (Algorithm 1 line 6; self-attention and softmax equations of Section 3.1).
 * For each selected row the whole logit row is formed, then its maximum, the
 * exponentials, their sum, and the weighted sum of value rows.
 *   q, k, v : [B, N, H, d]           q_idx : [B, M] or NULL (rows 0..M-1)
 *   kv_idx  : [B, M_kv] or NULL (all N keys; non-NULL is the "select Q and K"
 *             ablation, which restricts keys/values to the listed tokens)
 *   o       : [B, M, H, d] compact   lse : [B, H, M] = ln sum_j exp(s_j)
 *   p_out   : [B, H, M, Nk] softmax probabilities, or NULL
 */
void oracle_sparse_attn(const double *q, const double *k, const double *v,
                        const int32_t *q_idx, int M,
                        const int32_t *kv_idx, int M_kv,
                        double *o, double *lse, double *p_out,
                        int B, int H, int N, int N_kv, int d, double scale)
{
    /* N: tokens of q; N_kv: tokens of k and v (self-attention: N_kv == N; cross-attention of the
     * selected rows against another sequence, e.g. the text tokens: N_kv != N) */
    const int Nk = kv_idx ? M_kv : N_kv;
    if (scale == 0.0) scale = 1.0 / sqrt((double)d);
#pragma omp parallel
    {
        double *s = (double *)malloc((size_t)(Nk > 0 ? Nk : 1) * sizeof(double));
#pragma omp for collapse(2) schedule(dynamic, 1)
        for (int bh = 0; bh < B * H; ++bh) {
            for (int r = 0; r < M; ++r) {
                int b = bh / H, h = bh % H;
                int i = q_idx ? q_idx[(size_t)b * M + r] : r;
                const double *qi = q + (((size_t)b * N + i) * H + h) * d;
                double m = -INFINITY;
                for (int jj = 0; jj < Nk; ++jj) {
                    int j = kv_idx ? kv_idx[(size_t)b * M_kv + jj] : jj;
                    const double *kj = k + (((size_t)b * N_kv + j) * H + h) * d;
                    double dot = 0.0;
                    for (int c = 0; c < d; ++c) dot += qi[c] * kj[c];
                    s[jj] = dot * scale;
                    if (s[jj] > m) m = s[jj];
                }
                double Z = 0.0;
                for (int jj = 0; jj < Nk; ++jj) { s[jj] = exp(s[jj] - m); Z += s[jj]; }
                double *oi = o + (((size_t)b * M + r) * H + h) * d;
                for (int c = 0; c < d; ++c) oi[c] = 0.0;
                for (int jj = 0; jj < Nk; ++jj) {
                    int j = kv_idx ? kv_idx[(size_t)b * M_kv + jj] : jj;
                    const double *vj = v + (((size_t)b * N_kv + j) * H + h) * d;
                    double p = s[jj] / Z;
                    if (p_out) p_out[(((size_t)b * H + h) * M + r) * Nk + jj] = p;
                    for (int c = 0; c < d; ++c) oi[c] += p * vj[c];
                }
                if (lse) lse[((size_t)b * H + h) * M + r] = m + log(Z);
            }
        }
        free(s);
    }
}

/* ---------------------------------------------------------- scatter / reuse
 * X_out[I_sel] <- computed rows; X_out[I_remain] keeps the cached row
 * (Algorithm 1 lines 6-7).  `cache` [B, N, R] is updated in place; every row
 * not listed in idx is left untouched.
 */
void oracle_scatter_reuse(double *cache, const double *rows, const int32_t *idx,
                          int B, int N, int M, int R)
{
    for (int b = 0; b < B; ++b)
        for (int r = 0; r < M; ++r) {
            int i = idx[(size_t)b * M + r];
            memcpy(cache + ((size_t)b * N + i) * R, rows + ((size_t)b * M + r) * R,
                   (size_t)R * sizeof(double));
        }
}

/* lse cache [B, H, N] updated at the selected tokens from compact [B, H, M]. */
void oracle_scatter_lse(double *lse_cache, const double *lse_rows, const int32_t *idx,
                        int B, int H, int N, int M)
{
    for (int b = 0; b < B; ++b)
        for (int h = 0; h < H; ++h)
            for (int r = 0; r < M; ++r)
                lse_cache[((size_t)b * H + h) * N + idx[(size_t)b * M + r]] =
                    lse_rows[((size_t)b * H + h) * M + r];
}

/*
 * Linear layer on the selected rows (Algorithm 1 lines 4-5 and Section 3.2, "the same strategy
 * applies to the other layers of the block"): y[b, i, :] = x[b, i, :] W^T + bias for the listed
 * rows i = idx[b, r]; every other row of y keeps what it held (the cached result).  W is
 * [N_out, K] (out features x in features).  idx == NULL: all N rows.  Plain triple loop.
 * compact_in: x is [B, M, K] and its row r belongs to token idx[b, r] (the output of an earlier layer
 * that was computed on the selected rows only).  gelu: y = GELU(x W^T + bias) with the exact (erf)
 * definition GELU(u) = u/2 (1 + erf(u / sqrt 2)), the activation between the two MLP layers.
 */
void oracle_gathered_linear(const double *x, const int32_t *idx, int M, const double *w,
                            const double *bias, double *y, int B, int N, int K, int N_out,
                            int compact_in, int gelu)
{
    const int rows = idx ? M : N;
#pragma omp parallel for collapse(2) schedule(static)
    for (int b = 0; b < B; ++b)
        for (int r = 0; r < rows; ++r) {
            const int i = idx ? idx[(size_t)b * M + r] : r;
            const double *xr = compact_in ? x + ((size_t)b * M + r) * K : x + ((size_t)b * N + i) * K;
            double *yr = y + ((size_t)b * N + i) * N_out;
            for (int n = 0; n < N_out; ++n) {
                double acc = bias ? bias[n] : 0.0;
                const double *wr = w + (size_t)n * K;
                for (int c = 0; c < K; ++c) acc += xr[c] * wr[c];
                yr[n] = gelu ? 0.5 * acc * (1.0 + erf(acc * 0.70710678118654752440)) : acc;
            }
        }
}

/*
 * Layer normalisation of token rows followed by a per-batch-element modulation, the element-wise step in front
 * of every layer group of a compute block (Section 3.2: the layers of a block other than self-attention act on
 * each token by itself, so they are evaluated for the selected tokens only):
 *     y[r, :] = (x[r, :] - mean_r) / sqrt(var_r + eps) * (1 + scale[b, :]) + shift[b, :]
 * with the biased variance over the D channels and no learned affine; scale / shift NULL: plain normalisation.
 * x, y : [B, R, D] (R rows per batch element, whatever tokens they belong to); scale, shift : [B, D].
 */
void oracle_layernorm_modulate(const double *x, const double *scale, const double *shift, double *y,
                               int B, int R, int D, double eps)
{
    for (int b = 0; b < B; ++b)
        for (int r = 0; r < R; ++r) {
            const double *xr = x + ((size_t)b * R + r) * D;
            double *yr = y + ((size_t)b * R + r) * D;
            double mean = 0.0, var = 0.0;
            for (int c = 0; c < D; ++c) mean += xr[c];
            mean /= (double)D;
            for (int c = 0; c < D; ++c) var += (xr[c] - mean) * (xr[c] - mean);
            var /= (double)D;
            const double rstd = 1.0 / sqrt(var + eps);
            for (int c = 0; c < D; ++c) {
                double v = (xr[c] - mean) * rstd;
                if (scale) v *= 1.0 + scale[(size_t)b * D + c];
                if (shift) v += shift[(size_t)b * D + c];
                yr[c] = v;
            }
        }
}

/* floor(theta * N_sel) in integer arithmetic from a permille budget [R9]. */
int oracle_budget_to_k(int n_sel, int theta_permille)
{
    return (int)(((int64_t)n_sel * theta_permille) / 1000);
}
