// extern "C" entry points of the astraea library: argument validation on the host, then the
// kernel launchers.  No C++ exception crosses this boundary.
#include <stdarg.h>
#include <string.h>

#include <new>

#include "common.cuh"

namespace astraea {

static thread_local char g_err[512] = "";

void set_error(const char *fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
}

int32_t fail(int32_t code, const char *fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
    return code;
}

int32_t check_launch(const char *what) {
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return fail(ASTRAEA_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
    return ASTRAEA_OK;
}

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

void *tensor_map_encoder() {
    static void *const fn = [] {                   // function-local static: initialised once, thread-safe
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            ptr = nullptr;
        return ptr;
    }();
    return fn;
}

int sm_count() {
    static int cached[kMaxDevices] = {};
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return 148;
    int n = __atomic_load_n(&cached[dev], __ATOMIC_RELAXED);
    if (n > 0) return n;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) return 148;
    if (n > kMaxSMs) n = kMaxSMs;
    __atomic_store_n(&cached[dev], n, __ATOMIC_RELAXED);
    return n;
}

}  // namespace astraea

using namespace astraea;

#define REQUIRE(cond, ...) do { if (!(cond)) return fail(ASTRAEA_ERR_INVALID_ARG, __VA_ARGS__); } while (0)

extern "C" {

const char *astraea_last_error(void) { return g_err; }
const char *astraea_version(void) { return "astraea-b200 0.1 (sm_100a)"; }

int32_t astraea_budget_to_k(int n_sel, int theta_permille) {
    if (n_sel < 0 || theta_permille < 0 || theta_permille > 1000) return ASTRAEA_ERR_INVALID_ARG;
    return (int32_t)(((int64_t)n_sel * theta_permille) / 1000);
}

size_t astraea_workspace_bytes(int op, int B, int H, int N, int M, int d) {
    switch (op) {
    case ASTRAEA_OP_SELECT: return select_workspace_bytes(B, N);
    case ASTRAEA_OP_SPARSE_ATTN: return attn_workspace_bytes(B, H, N, M, d);
    case ASTRAEA_OP_SPARSE_ATTN_KV: return attn_kv_workspace_bytes(B, H, M, d);
    case ASTRAEA_OP_STEP: return attn_workspace_bytes(B, H, N, M, d) + align_up(select_workspace_bytes(B, N), 256);
    case ASTRAEA_OP_GATHERED_LINEAR: return linear_workspace_bytes();
    case ASTRAEA_OP_LAYERNORM: return 256;
    default: return 0;
    }
}

int32_t astraea_score(const void *x_cur, const void *x_ref, const float *lse, const int32_t *n_skip,
                      float *score, int B, int N, int N_sel, int D, int H,
                      float w_alpha, float w_beta, int delta_mode, int lse_mode, void *stream)
{
    REQUIRE(B > 0 && N > 0 && D > 0 && H > 0, "astraea_score: B, N, D, H must be positive");
    REQUIRE(N_sel >= 0 && N_sel <= N, "astraea_score: N_sel=%d outside [0, N=%d]", N_sel, N);
    REQUIRE(D % 8 == 0, "astraea_score: D=%d must be a multiple of 8 (16-byte rows)", D);
    REQUIRE(x_cur && x_ref && score, "astraea_score: null x_cur, x_ref or score");
    REQUIRE(aligned16(x_cur) && aligned16(x_ref), "astraea_score: x_cur / x_ref must be 16-byte aligned");
    if (delta_mode < 0 || delta_mode > 2 || lse_mode < 0 || lse_mode > 1)
        return fail(ASTRAEA_ERR_UNSUPPORTED, "astraea_score: unknown delta_mode %d or lse_mode %d", delta_mode, lse_mode);
    return launch_score(x_cur, x_ref, lse, n_skip, score, B, N, N_sel, D, H, w_alpha, w_beta, delta_mode,
                        lse_mode, (cudaStream_t)stream);
}

int32_t astraea_score_partial(const void *x_cur, const void *x_ref, const float *lse, float *part,
                              int B, int N, int N_sel, int D_local, int H_local, int delta_mode, int lse_mode, void *stream)
{
    REQUIRE(B > 0 && N > 0 && D_local > 0 && H_local > 0, "astraea_score_partial: B, N, D_local, H_local must be positive");
    REQUIRE(N_sel >= 0 && N_sel <= N, "astraea_score_partial: N_sel=%d outside [0, N=%d]", N_sel, N);
    REQUIRE(D_local % 8 == 0, "astraea_score_partial: D_local=%d must be a multiple of 8 (16-byte rows)", D_local);
    REQUIRE(x_cur && x_ref && part, "astraea_score_partial: null x_cur, x_ref or part");
    REQUIRE(aligned16(x_cur) && aligned16(x_ref), "astraea_score_partial: x_cur / x_ref must be 16-byte aligned");
    if (delta_mode < 0 || delta_mode > 2 || lse_mode < 0 || lse_mode > 1)
        return fail(ASTRAEA_ERR_UNSUPPORTED, "astraea_score_partial: unknown delta_mode %d or lse_mode %d", delta_mode, lse_mode);
    return launch_score(x_cur, x_ref, lse, nullptr, nullptr, B, N, N_sel, D_local, H_local, 0.f, 0.f, delta_mode, lse_mode,
                        (cudaStream_t)stream, part);
}

int32_t astraea_score_combine(const float *part, const int32_t *n_skip, float *score, int B, int N_sel, int D, int H,
                              int has_lse, float w_alpha, float w_beta, void *stream)
{
    REQUIRE(B > 0 && N_sel >= 0 && D > 0 && H > 0, "astraea_score_combine: bad sizes");
    REQUIRE((part && score) || N_sel == 0, "astraea_score_combine: null part or score");
    return launch_score_combine(part, n_skip, score, B, N_sel, D, H, has_lse ? 1 : 0, w_alpha, w_beta, (cudaStream_t)stream);
}

int32_t astraea_select(const float *score, int B, int N_sel, int k, int n_always,
                       int32_t *idx_sel, int32_t *idx_rem, int32_t *n_skip,
                       void *workspace, size_t workspace_bytes, void *stream)
{
    REQUIRE(B > 0 && N_sel >= 0 && n_always >= 0, "astraea_select: bad sizes");
    REQUIRE(k >= 0 && k <= N_sel, "astraea_select: k=%d outside [0, N_sel=%d]", k, N_sel);
    REQUIRE(score || N_sel == 0, "astraea_select: null score");
    REQUIRE(idx_sel || (k + n_always) == 0, "astraea_select: null idx_sel");
    if (workspace_bytes < select_workspace_bytes(B, N_sel) || !workspace)
        return fail(ASTRAEA_ERR_WORKSPACE_TOO_SMALL, "astraea_select: workspace of %zu bytes, need %zu",
                    workspace_bytes, select_workspace_bytes(B, N_sel));
    REQUIRE(aligned16(workspace), "astraea_select: workspace must be 16-byte aligned");
    return launch_select(score, B, N_sel, k, n_always, idx_sel, idx_rem, n_skip, workspace, (cudaStream_t)stream);
}

static int32_t sparse_attn_entry(const char *fn, int N_kv, const void *q, const void *k, const void *v,
                            int64_t q_sb, int64_t q_sh, int64_t q_sn,
                            int64_t k_sb, int64_t k_sh, int64_t k_sn,
                            int64_t v_sb, int64_t v_sh, int64_t v_sn,
                            const int32_t *q_idx, int M, const int32_t *kv_idx, int M_kv,
                            void *out, float *lse_out,
                            int B, int H, int N, int d, float scale, uint32_t flags,
                            void *workspace, size_t workspace_bytes, void *stream)
{
    REQUIRE(B > 0 && H > 0 && N > 0 && d > 0 && N_kv >= 0, "%s: B, H, N, d must be positive", fn);
    REQUIRE(!kv_idx || (M_kv > 0 && M_kv <= N), "%s: M_kv=%d outside [1, N=%d]", fn, M_kv, N);
    REQUIRE(M >= 0 && M <= N, "%s: M=%d outside [0, N=%d]", fn, M, N);
    if (d != 64 && d != 72 && d != 128)
        return fail(ASTRAEA_ERR_UNSUPPORTED, "%s: head_dim %d not in {64, 72, 128}", fn, d);
    if (flags & ~(ASTRAEA_ATTN_COMPACT_OUT | ASTRAEA_ATTN_SMALL_CTAS | ASTRAEA_ATTN_WHOLE_KEYS)) return fail(ASTRAEA_ERR_UNSUPPORTED, "%s: unknown flags 0x%x", fn, flags);
    REQUIRE(q && k && v && out, "%s: null q, k, v or out", fn);
    REQUIRE(aligned16(q) && aligned16(k) && aligned16(v) && aligned16(out), "%s: q, k, v, out must be 16-byte aligned", fn);
    REQUIRE(q_sn % 8 == 0 && k_sn % 8 == 0 && v_sn % 8 == 0 && q_sh % 8 == 0 && k_sh % 8 == 0 && v_sh % 8 == 0 &&
            q_sb % 8 == 0 && k_sb % 8 == 0 && v_sb % 8 == 0,
            "%s: strides must be multiples of 8 elements (16 bytes)", fn);
    REQUIRE(q_sn >= d && k_sn >= d && v_sn >= d && q_sh > 0 && k_sh > 0 && v_sh > 0 && q_sb >= 0 && k_sb >= 0 && v_sb >= 0,
            "%s: strides must be positive and token stride >= head_dim", fn);
    REQUIRE(scale >= 0.f, "%s: scale must be >= 0 (0 selects 1/sqrt(d))", fn);
    // without kv_idx the error word is all a launch needs; what lies behind it lets the launch split its last round of CTAs
    const size_t ws_need = kv_idx ? attn_kv_workspace_bytes(B, H, M_kv, d) : 256;
    if (!workspace || workspace_bytes < ws_need)
        return fail(ASTRAEA_ERR_WORKSPACE_TOO_SMALL, "%s: workspace of %zu bytes, need %zu", fn,
                    workspace_bytes, ws_need);
    REQUIRE((reinterpret_cast<uintptr_t>(workspace) & 255u) == 0, "%s: workspace must be 256-byte aligned", fn);
    if (M == 0) return ASTRAEA_OK;
    AttnArgs a;
    a.q = q; a.k = k; a.v = v;
    a.q_sb = q_sb; a.q_sh = q_sh; a.q_sn = q_sn;
    a.k_sb = k_sb; a.k_sh = k_sh; a.k_sn = k_sn;
    a.v_sb = v_sb; a.v_sh = v_sh; a.v_sn = v_sn;
    a.q_idx = q_idx; a.M = M; a.out = out; a.lse_out = lse_out;
    a.B = B; a.H = H; a.N = N; a.d = d;
    a.scale = (scale == 0.f) ? 1.0f / sqrtf((float)d) : scale;
    a.flags = flags;
    a.err_word = reinterpret_cast<int *>(workspace);
    a.N_tok = N;
    if (N_kv > 0) a.N = N_kv;          // keys and values of another sequence: N stays the token count of q / out
    if (kv_idx) return launch_sparse_attn_kv(a, kv_idx, M_kv, workspace, (cudaStream_t)stream);
    if (workspace_bytes > 256) { a.split_ws = static_cast<char *>(workspace) + 256; a.split_ws_bytes = workspace_bytes - 256; }
    return launch_sparse_attn(a, (cudaStream_t)stream);
}

int32_t astraea_sparse_attn(const void *q, const void *k, const void *v,
                            int64_t q_sb, int64_t q_sh, int64_t q_sn,
                            int64_t k_sb, int64_t k_sh, int64_t k_sn,
                            int64_t v_sb, int64_t v_sh, int64_t v_sn,
                            const int32_t *q_idx, int M, const int32_t *kv_idx, int M_kv,
                            void *out, float *lse_out,
                            int B, int H, int N, int d, float scale, uint32_t flags,
                            void *workspace, size_t workspace_bytes, void *stream)
{
    return sparse_attn_entry("astraea_sparse_attn", 0, q, k, v, q_sb, q_sh, q_sn, k_sb, k_sh, k_sn, v_sb, v_sh, v_sn,
                             q_idx, M, kv_idx, M_kv, out, lse_out, B, H, N, d, scale, flags, workspace, workspace_bytes, stream);
}

int32_t astraea_sparse_attn_plan(int B, int H, int N, int M, int d, uint32_t flags, size_t workspace_bytes,
                                 int32_t *small_ctas, int32_t *split_units, int32_t *split)
{
    REQUIRE(B > 0 && H > 0 && N > 0 && M >= 0 && M <= N, "astraea_sparse_attn_plan: bad sizes");
    REQUIRE(small_ctas && split_units && split, "astraea_sparse_attn_plan: null result pointer");
    if (d != 64 && d != 72 && d != 128) return fail(ASTRAEA_ERR_UNSUPPORTED, "astraea_sparse_attn_plan: head_dim %d not in {64, 72, 128}", d);
    AttnArgs a = {};
    a.B = B; a.H = H; a.N = N; a.N_tok = N; a.M = M; a.d = d; a.flags = flags;
    static char nowhere;                       // never dereferenced: the plan only asks whether there is room
    if (workspace_bytes > 256) { a.split_ws = &nowhere; a.split_ws_bytes = workspace_bytes - 256; }
    int s = 0, u = 0, k = 1;
    if (M > 0) attn_plan(a, &s, &u, &k);
    *small_ctas = s; *split_units = u; *split = k;
    return ASTRAEA_OK;
}

int32_t astraea_sparse_cross_attn(const void *q, const void *k, const void *v,
                                  int64_t q_sb, int64_t q_sh, int64_t q_sn,
                                  int64_t k_sb, int64_t k_sh, int64_t k_sn,
                                  int64_t v_sb, int64_t v_sh, int64_t v_sn,
                                  const int32_t *q_idx, int M, void *out, float *lse_out,
                                  int B, int H, int N, int N_kv, int d, float scale, uint32_t flags,
                                  void *workspace, size_t workspace_bytes, void *stream)
{
    REQUIRE(N_kv > 0, "astraea_sparse_cross_attn: N_kv=%d must be positive", N_kv);
    return sparse_attn_entry("astraea_sparse_cross_attn", N_kv, q, k, v, q_sb, q_sh, q_sn, k_sb, k_sh, k_sn, v_sb, v_sh, v_sn,
                             q_idx, M, nullptr, 0, out, lse_out, B, H, N, d, scale, flags, workspace, workspace_bytes, stream);
}

int32_t astraea_sparse_attn_noalloc(const void *q, const void *k, const void *v,
                                    int64_t q_sb, int64_t q_sh, int64_t q_sn,
                                    int64_t k_sb, int64_t k_sh, int64_t k_sn,
                                    int64_t v_sb, int64_t v_sh, int64_t v_sn,
                                    const int32_t *q_idx, int M, const int32_t *kv_idx, int M_kv,
                                    void *out, float *lse_out,
                                    int B, int H, int N, int d, float scale, uint32_t flags, void *stream)
{
    // the scratch is the library's own fixed array: resolve its address on this device (first call: set-up), clear
    // the error word the last call may have left, then run the ordinary entry with it as the workspace
    void *scratch = nullptr;
    int32_t rc = noalloc_scratch_address(&scratch);
    if (rc != ASTRAEA_OK) return rc;
    cudaError_t e = cudaMemsetAsync(scratch, 0, 256, (cudaStream_t)stream);
    if (e != cudaSuccess) return fail(ASTRAEA_ERR_CUDA, "astraea_sparse_attn_noalloc: clearing the scratch failed: %s", cudaGetErrorString(e));
    return sparse_attn_entry("astraea_sparse_attn_noalloc", 0, q, k, v, q_sb, q_sh, q_sn, k_sb, k_sh, k_sn, v_sb, v_sh, v_sn,
                             q_idx, M, kv_idx, M_kv, out, lse_out, B, H, N, d, scale, flags, scratch,
                             ASTRAEA_NOALLOC_SCRATCH_BYTES, stream);
}

int32_t astraea_scatter_reuse(void *cache, const void *rows, const int32_t *idx,
                              int B, int N, int M, int row_elems, uint32_t flags, void *err_workspace, void *stream)
{
    REQUIRE(B > 0 && N > 0 && row_elems > 0, "astraea_scatter_reuse: B, N, row_elems must be positive");
    REQUIRE(M >= 0 && M <= N, "astraea_scatter_reuse: M=%d outside [0, N=%d]", M, N);
    REQUIRE(row_elems % 8 == 0, "astraea_scatter_reuse: row_elems=%d must be a multiple of 8", row_elems);
    if (flags & ~ASTRAEA_SCATTER_SRC_FULL) return fail(ASTRAEA_ERR_UNSUPPORTED, "astraea_scatter_reuse: unknown flags 0x%x", flags);
    if (M == 0) return ASTRAEA_OK;
    REQUIRE(cache && rows && idx, "astraea_scatter_reuse: null cache, rows or idx");
    REQUIRE(aligned16(cache) && aligned16(rows), "astraea_scatter_reuse: cache / rows must be 16-byte aligned");
    REQUIRE((reinterpret_cast<uintptr_t>(err_workspace) & 3u) == 0, "astraea_scatter_reuse: err_workspace must be 4-byte aligned");
    return launch_scatter(cache, rows, idx, B, N, M, row_elems, flags, reinterpret_cast<int *>(err_workspace), (cudaStream_t)stream);
}

int32_t astraea_gathered_linear_residual(const void *x, const int32_t *idx, int M, const void *w, const void *bias,
                                         const void *residual, const void *gate,
                                         void *y, int B, int N, int K, int N_out, uint32_t flags,
                                         void *workspace, size_t workspace_bytes, void *stream)
{
    REQUIRE(B > 0 && N > 0 && K > 0 && N_out > 0, "astraea_gathered_linear: B, N, K, N_out must be positive");
    REQUIRE(!idx || (M >= 0 && M <= N), "astraea_gathered_linear: M=%d outside [0, N=%d]", M, N);
    REQUIRE(K % 64 == 0, "astraea_gathered_linear: K=%d must be a multiple of 64", K);
    REQUIRE(N_out % 8 == 0, "astraea_gathered_linear: N_out=%d must be a multiple of 8", N_out);
    if (flags & ~(ASTRAEA_LINEAR_COMPACT_OUT | ASTRAEA_LINEAR_COMPACT_IN | ASTRAEA_LINEAR_GELU | ASTRAEA_LINEAR_COMPACT_RES))
        return fail(ASTRAEA_ERR_UNSUPPORTED, "astraea_gathered_linear: unknown flags 0x%x", flags);
    REQUIRE(!(flags & (ASTRAEA_LINEAR_COMPACT_OUT | ASTRAEA_LINEAR_COMPACT_IN | ASTRAEA_LINEAR_COMPACT_RES)) || idx,
            "astraea_gathered_linear: compact rows need an index list");
    REQUIRE(!(flags & ASTRAEA_LINEAR_COMPACT_RES) || residual, "astraea_gathered_linear: ASTRAEA_LINEAR_COMPACT_RES without a residual");
    if (!workspace || workspace_bytes < linear_workspace_bytes())
        return fail(ASTRAEA_ERR_WORKSPACE_TOO_SMALL, "astraea_gathered_linear: workspace of %zu bytes, need %zu",
                    workspace_bytes, linear_workspace_bytes());
    REQUIRE((reinterpret_cast<uintptr_t>(workspace) & 255u) == 0, "astraea_gathered_linear: workspace must be 256-byte aligned");
    if (idx && M == 0) return ASTRAEA_OK;
    REQUIRE(x && w && y, "astraea_gathered_linear: null x, w or y");
    REQUIRE(aligned16(x) && aligned16(w) && aligned16(y) && aligned16(bias) && aligned16(residual) && aligned16(gate),
            "astraea_gathered_linear: x, w, bias, residual, gate, y must be 16-byte aligned");
    return launch_gathered_linear(x, idx, M, w, bias, y, B, N, K, N_out, flags, reinterpret_cast<int *>(workspace),
                                  (cudaStream_t)stream, residual, gate);
}

int32_t astraea_gathered_linear(const void *x, const int32_t *idx, int M, const void *w, const void *bias,
                                void *y, int B, int N, int K, int N_out, uint32_t flags,
                                void *workspace, size_t workspace_bytes, void *stream)
{
    if (flags & ASTRAEA_LINEAR_COMPACT_RES) return fail(ASTRAEA_ERR_UNSUPPORTED, "astraea_gathered_linear: unknown flags 0x%x", flags);
    return astraea_gathered_linear_residual(x, idx, M, w, bias, nullptr, nullptr, y, B, N, K, N_out, flags, workspace,
                                            workspace_bytes, stream);
}

int32_t astraea_layernorm_modulate(const void *x, const int32_t *idx, int M, const void *scale, const void *shift,
                                   void *y, int B, int N, int D, float eps, uint32_t flags,
                                   void *err_workspace, void *stream)
{
    REQUIRE(B > 0 && N > 0 && D > 0, "astraea_layernorm_modulate: B, N, D must be positive");
    REQUIRE(D % 8 == 0, "astraea_layernorm_modulate: D=%d must be a multiple of 8", D);
    REQUIRE(!idx || (M >= 0 && M <= N), "astraea_layernorm_modulate: M=%d outside [0, N=%d]", M, N);
    REQUIRE(eps >= 0.f, "astraea_layernorm_modulate: eps must be >= 0");
    if (flags & ~(ASTRAEA_LN_COMPACT_IN | ASTRAEA_LN_COMPACT_OUT))
        return fail(ASTRAEA_ERR_UNSUPPORTED, "astraea_layernorm_modulate: unknown flags 0x%x", flags);
    REQUIRE(!flags || idx, "astraea_layernorm_modulate: compact rows need an index list");
    if (idx && M == 0) return ASTRAEA_OK;
    REQUIRE(x && y, "astraea_layernorm_modulate: null x or y");
    REQUIRE(aligned16(x) && aligned16(y) && aligned16(scale) && aligned16(shift), "astraea_layernorm_modulate: pointers must be 16-byte aligned");
    REQUIRE((reinterpret_cast<uintptr_t>(err_workspace) & 3u) == 0, "astraea_layernorm_modulate: err_workspace must be 4-byte aligned");
    return launch_layernorm_modulate(x, idx, M, scale, shift, y, B, N, D, eps, flags, reinterpret_cast<int *>(err_workspace),
                                     (cudaStream_t)stream);
}

// ------------------------------------------------------------------ a whole compute block
// workspace: [256 bytes: error word | gathered keys and values of the SelectQ&K variant, or the key shares of a split
//             self-attention launch] [select scratch]
//            [5 token-sized buffers] [hidden-sized buffer]
// (the first part is laid out as the workspace of astraea_sparse_attn with kv_idx, so that every call of the block
// shares the one error word at the very start)
static size_t block_buffer_bytes(int B, int N, int width) { return align_up((size_t)B * N * width * 2, 256); }
// the head of the block's workspace serves the self-attention: gathered keys / values (SelectQ&K) or the key shares of a split launch
static size_t block_attn_region_bytes(int B, int H, int N, int d)
{
    const size_t kv = attn_kv_workspace_bytes(B, H, N, d), plain = attn_workspace_bytes(B, H, N, N, d);
    return align_up(kv > plain ? kv : plain, 256);
}

size_t astraea_block_workspace_bytes(int B, int H, int N, int d, int hidden)
{
    if (B <= 0 || H <= 0 || N <= 0 || d <= 0 || hidden <= 0) return 0;
    return block_attn_region_bytes(B, H, N, d) + align_up(select_workspace_bytes(B, N), 256) +
           5 * block_buffer_bytes(B, N, H * d) + block_buffer_bytes(B, N, hidden);
}

int32_t astraea_block_step(const void *x, const astraea_block_weights *w, const astraea_block_state *st,
                           const void *text_k, const void *text_v, int N_text,
                           float *score, int32_t *idx_sel, int32_t *idx_rem,
                           int B, int H, int N, int N_sel, int d, int k_keep,
                           float w_alpha, float w_beta, int delta_mode, int lse_mode, float eps, uint32_t flags,
                           void *workspace, size_t workspace_bytes, void *stream)
{
    REQUIRE(x && w && st, "astraea_block_step: null x, weights or state");
    REQUIRE(B > 0 && H > 0 && N > 0 && d > 0 && N_text > 0, "astraea_block_step: B, H, N, d, N_text must be positive");
    REQUIRE(N_sel >= 0 && N_sel <= N, "astraea_block_step: N_sel=%d outside [0, N=%d]", N_sel, N);
    REQUIRE(k_keep >= 0 && k_keep <= N_sel, "astraea_block_step: k_keep=%d outside [0, N_sel=%d]", k_keep, N_sel);
    if (flags & ~(ASTRAEA_BLOCK_REUSE_SELECTION | ASTRAEA_BLOCK_SELECT_QK))
        return fail(ASTRAEA_ERR_UNSUPPORTED, "astraea_block_step: unknown flags 0x%x", flags);
    const int D = H * d, hidden = w->hidden;
    REQUIRE(D % 64 == 0 && hidden > 0 && hidden % 64 == 0, "astraea_block_step: D=%d and hidden=%d must be multiples of 64", D, hidden);
    REQUIRE(w->wq && w->wk && w->wv && w->wo && w->wq2 && w->wo2 && w->w1 && w->w2, "astraea_block_step: null weight matrix");
    REQUIRE(st->x_ref && st->lse_cache && st->y_cache, "astraea_block_step: null state buffer");
    REQUIRE(text_k && text_v, "astraea_block_step: null text keys / values");
    const size_t need = astraea_block_workspace_bytes(B, H, N, d, hidden);
    if (!workspace || workspace_bytes < need)
        return fail(ASTRAEA_ERR_WORKSPACE_TOO_SMALL, "astraea_block_step: workspace of %zu bytes, need %zu", workspace_bytes, need);
    REQUIRE((reinterpret_cast<uintptr_t>(workspace) & 255u) == 0, "astraea_block_step: workspace must be 256-byte aligned");
    const int n_always = N - N_sel, M = k_keep + n_always;
    REQUIRE(score && (idx_sel || M == 0), "astraea_block_step: null score or idx_sel");
    char *ws = reinterpret_cast<char *>(workspace);
    void *err = ws;                                     // the error word of every call below
    char *p = ws + block_attn_region_bytes(B, H, N, d);
    void *sel_ws = p; p += align_up(select_workspace_bytes(B, N), 256);
    const size_t tb = block_buffer_bytes(B, N, D);
    void *bufA = p, *bufQ = p + tb, *bufK = p + 2 * tb, *bufV = p + 3 * tb, *bufO = p + 4 * tb, *bufU = p + 5 * tb;
    const bool select_qk = (flags & ASTRAEA_BLOCK_SELECT_QK) != 0;
    int32_t rc = ASTRAEA_OK;
    if (!(flags & ASTRAEA_BLOCK_REUSE_SELECTION)) {
        rc = astraea_score(x, st->x_ref, st->lse_cache, st->n_skip, score, B, N, N_sel, D, H, w_alpha, w_beta, delta_mode, lse_mode, stream);
        if (rc == ASTRAEA_OK)
            rc = astraea_select(score, B, N_sel, k_keep, n_always, idx_sel, idx_rem, st->n_skip, sel_ws, select_workspace_bytes(B, N), stream);
        if (rc != ASTRAEA_OK) return rc;
    }
    if (M == 0) return ASTRAEA_OK;
    const int64_t sb = (int64_t)N * D, sh = d, sn = D;
    const int64_t tsb = (int64_t)N_text * D;
    // self-attention group: keys / values from all tokens, everything else on the selected rows
    rc = astraea_layernorm_modulate(x, nullptr, 0, w->s1, w->t1, bufA, B, N, D, eps, 0u, err, stream);
    // (SelectQ&K: keys and values of the selected tokens only, so only their rows are projected)
    const int32_t *kv_rows = select_qk ? idx_sel : nullptr;
    if (rc == ASTRAEA_OK) rc = astraea_gathered_linear(bufA, kv_rows, M, w->wk, w->bk, bufK, B, N, D, D, 0u, err, 256, stream);
    if (rc == ASTRAEA_OK) rc = astraea_gathered_linear(bufA, kv_rows, M, w->wv, w->bv, bufV, B, N, D, D, 0u, err, 256, stream);
    if (rc == ASTRAEA_OK) rc = astraea_gathered_linear(bufA, idx_sel, M, w->wq, w->bq, bufQ, B, N, D, D, 0u, err, 256, stream);
    if (rc == ASTRAEA_OK && !select_qk)
        rc = astraea_sparse_attn(bufQ, bufK, bufV, sb, sh, sn, sb, sh, sn, sb, sh, sn, idx_sel, M, nullptr, 0, bufO, st->lse_cache,
                                 B, H, N, d, 0.f, 0u, ws, block_attn_region_bytes(B, H, N, d), stream);
    if (rc == ASTRAEA_OK && select_qk)       // the listed key / value rows are gathered into the head of the workspace
        rc = astraea_sparse_attn(bufQ, bufK, bufV, sb, sh, sn, sb, sh, sn, sb, sh, sn, idx_sel, M, idx_sel, M, bufO, st->lse_cache,
                                 B, H, N, d, 0.f, 0u, ws, attn_kv_workspace_bytes(B, H, N, d), stream);
    // x1 (compact, over the dead keys) = x[I] + g1 * (attention rows Wo^T + bo)
    if (rc == ASTRAEA_OK)
        rc = astraea_gathered_linear_residual(bufO, idx_sel, M, w->wo, w->bo, x, w->g1, bufK, B, N, D, D, ASTRAEA_LINEAR_COMPACT_OUT, err, 256, stream);
    // cross-attention group on the compact rows
    if (rc == ASTRAEA_OK)
        rc = astraea_layernorm_modulate(bufK, idx_sel, M, nullptr, nullptr, bufA, B, N, D, eps, ASTRAEA_LN_COMPACT_IN | ASTRAEA_LN_COMPACT_OUT, err, stream);
    if (rc == ASTRAEA_OK) rc = astraea_gathered_linear(bufA, idx_sel, M, w->wq2, w->bq2, bufQ, B, N, D, D, ASTRAEA_LINEAR_COMPACT_IN, err, 256, stream);
    if (rc == ASTRAEA_OK)
        rc = astraea_sparse_cross_attn(bufQ, text_k, text_v, sb, sh, sn, tsb, sh, sn, tsb, sh, sn, idx_sel, M, bufV, nullptr, B, H, N, N_text, d,
                                       0.f, ASTRAEA_ATTN_COMPACT_OUT, err, 256, stream);
    if (rc == ASTRAEA_OK)       // x2 (compact, over the dead attention rows) = x1 + cross rows Wo2^T + bo2
        rc = astraea_gathered_linear_residual(bufV, idx_sel, M, w->wo2, w->bo2, bufK, nullptr, bufO, B, N, D, D,
                                              ASTRAEA_LINEAR_COMPACT_IN | ASTRAEA_LINEAR_COMPACT_OUT | ASTRAEA_LINEAR_COMPACT_RES, err, 256, stream);
    // MLP group: the hidden activations exist for the selected rows only; the result lands in the block's cache
    if (rc == ASTRAEA_OK)
        rc = astraea_layernorm_modulate(bufO, idx_sel, M, w->s3, w->t3, bufA, B, N, D, eps, ASTRAEA_LN_COMPACT_IN | ASTRAEA_LN_COMPACT_OUT, err, stream);
    if (rc == ASTRAEA_OK)
        rc = astraea_gathered_linear(bufA, idx_sel, M, w->w1, w->b1, bufU, B, N, D, hidden,
                                     ASTRAEA_LINEAR_COMPACT_IN | ASTRAEA_LINEAR_COMPACT_OUT | ASTRAEA_LINEAR_GELU, err, 256, stream);
    if (rc == ASTRAEA_OK)
        rc = astraea_gathered_linear_residual(bufU, idx_sel, M, w->w2, w->b2, bufO, w->g3, st->y_cache, B, N, hidden, D,
                                              ASTRAEA_LINEAR_COMPACT_IN | ASTRAEA_LINEAR_COMPACT_RES, err, 256, stream);
    // the reference inputs of the tokens that were computed become the current inputs
    if (rc == ASTRAEA_OK && !(flags & ASTRAEA_BLOCK_REUSE_SELECTION))
        rc = astraea_scatter_reuse(st->x_ref, x, idx_sel, B, N, M, D, ASTRAEA_SCATTER_SRC_FULL, err, stream);
    return rc;
}

int32_t astraea_step(const void *x_cur, void *x_ref, float *lse_cache, int32_t *n_skip,
                     const void *q, const void *k, const void *v, void *out_cache,
                     float *score, int32_t *idx_sel, int32_t *idx_rem,
                     int B, int H, int N, int N_sel, int d, int k_keep,
                     float w_alpha, float w_beta, int delta_mode, int lse_mode,
                     void *workspace, size_t workspace_bytes, void *stream)
{
    REQUIRE(N_sel >= 0 && N_sel <= N, "astraea_step: N_sel=%d outside [0, N=%d]", N_sel, N);
    REQUIRE(k_keep >= 0 && k_keep <= N_sel, "astraea_step: k_keep=%d outside [0, N_sel=%d]", k_keep, N_sel);
    const int n_always = N - N_sel;
    const int M = k_keep + n_always;
    const int D = H * d;
    const size_t attn_ws = attn_workspace_bytes(B, H, N, M, d);
    if (!workspace || workspace_bytes < astraea_workspace_bytes(ASTRAEA_OP_STEP, B, H, N, M, d))
        return fail(ASTRAEA_ERR_WORKSPACE_TOO_SMALL, "astraea_step: workspace of %zu bytes, need %zu", workspace_bytes,
                    astraea_workspace_bytes(ASTRAEA_OP_STEP, B, H, N, M, d));
    REQUIRE(score && (idx_sel || M == 0), "astraea_step: null score or idx_sel");
    char *ws = reinterpret_cast<char *>(workspace);
    int32_t rc = astraea_score(x_cur, x_ref, lse_cache, n_skip, score, B, N, N_sel, D, H, w_alpha, w_beta,
                               delta_mode, lse_mode, stream);
    if (rc != ASTRAEA_OK) return rc;
    rc = astraea_select(score, B, N_sel, k_keep, n_always, idx_sel, idx_rem, n_skip, ws + attn_ws,
                        workspace_bytes - attn_ws, stream);
    if (rc != ASTRAEA_OK) return rc;
    const int64_t sb = (int64_t)N * D, sh = d, sn = D;
    rc = astraea_sparse_attn(q, k, v, sb, sh, sn, sb, sh, sn, sb, sh, sn, idx_sel, M, nullptr, 0, out_cache,
                             lse_cache, B, H, N, d, 0.f, 0u, ws, attn_ws, stream);
    if (rc != ASTRAEA_OK) return rc;
    // the reference inputs of the tokens that were computed become the current inputs
    return astraea_scatter_reuse(x_ref, x_cur, idx_sel, B, N, M, D, ASTRAEA_SCATTER_SRC_FULL, ws, stream);
}

int32_t astraea_selftest_wait(void *workspace, int limit_us, int32_t *gave_up, void *stream)
{
    REQUIRE(workspace, "astraea_selftest_wait: null workspace");
    REQUIRE(limit_us > 0 && limit_us <= 1000, "astraea_selftest_wait: limit_us=%d outside [1, 1000]", limit_us);
    return launch_wait_selftest(reinterpret_cast<int *>(workspace), (uint64_t)limit_us * 1000ull, gave_up, (cudaStream_t)stream);
}

int32_t astraea_poll_error(void *workspace, void *stream)
{
    REQUIRE(workspace, "astraea_poll_error: null workspace");
    int word = 0;
    cudaError_t e = cudaStreamSynchronize((cudaStream_t)stream);
    if (e == cudaSuccess) e = cudaMemcpy(&word, workspace, sizeof(int), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return fail(ASTRAEA_ERR_CUDA, "astraea_poll_error: %s", cudaGetErrorString(e));
    if (word != 0) cudaMemset(workspace, 0, sizeof(int));
    if (word == kErrTimeout) return fail(ASTRAEA_ERR_TIMEOUT, "a bounded device-side wait gave up");
    if (word == kErrBadIndex) return fail(ASTRAEA_ERR_BAD_INDEX, "an index list held an entry out of range or not strictly ascending");
    return ASTRAEA_OK;
}

// ------------------------------------------------------------------ a schedule of steps as one CUDA graph
struct astraea_schedule {
    cudaGraph_t graph;
    cudaGraphExec_t exec;
    int T;
};

void astraea_schedule_destroy(astraea_schedule *s)
{
    if (!s) return;
    if (s->exec) cudaGraphExecDestroy(s->exec);
    if (s->graph) cudaGraphDestroy(s->graph);
    delete s;
}

int32_t astraea_schedule_create(astraea_schedule **schedule, int T, const int32_t *k_keep,
                                const void *const *x_cur, const void *const *q, const void *const *k,
                                const void *const *v, void *x_ref, float *lse_cache, int32_t *n_skip,
                                void *out_cache, float *score, int32_t *idx_sel, int32_t *idx_rem,
                                int B, int H, int N, int N_sel, int d,
                                float w_alpha, float w_beta, int delta_mode, int lse_mode,
                                void *workspace, size_t workspace_bytes)
{
    REQUIRE(schedule, "astraea_schedule_create: null schedule pointer");
    *schedule = nullptr;
    REQUIRE(T > 0 && k_keep && x_cur && q && k && v, "astraea_schedule_create: T must be positive and the per-step arrays non-null");
    REQUIRE(N_sel >= 0 && N_sel <= N, "astraea_schedule_create: N_sel=%d outside [0, N=%d]", N_sel, N);
    for (int t = 0; t < T; ++t) {
        REQUIRE(k_keep[t] >= 0 && k_keep[t] <= N_sel, "astraea_schedule_create: k_keep[%d]=%d outside [0, N_sel=%d]", t, k_keep[t], N_sel);
        REQUIRE(x_cur[t] && q[t] && k[t] && v[t], "astraea_schedule_create: null input pointer at step %d", t);
    }
    if (!workspace || workspace_bytes < astraea_workspace_bytes(ASTRAEA_OP_STEP, B, H, N, N, d))
        return fail(ASTRAEA_ERR_WORKSPACE_TOO_SMALL, "astraea_schedule_create: workspace of %zu bytes, need %zu",
                    workspace_bytes, astraea_workspace_bytes(ASTRAEA_OP_STEP, B, H, N, N, d));
    astraea_schedule *s = new (std::nothrow) astraea_schedule();
    if (!s) return fail(ASTRAEA_ERR_CUDA, "astraea_schedule_create: out of host memory");
    s->graph = nullptr; s->exec = nullptr; s->T = T;
    cudaStream_t cap = nullptr;
    cudaError_t e = cudaStreamCreateWithFlags(&cap, cudaStreamNonBlocking);
    if (e != cudaSuccess) { delete s; return fail(ASTRAEA_ERR_CUDA, "astraea_schedule_create: %s", cudaGetErrorString(e)); }
    // a thread-local capture: other threads of the process may keep using CUDA meanwhile
    e = cudaStreamBeginCapture(cap, cudaStreamCaptureModeThreadLocal);
    int32_t rc = ASTRAEA_OK;
    if (e == cudaSuccess) {
        for (int t = 0; t < T && rc == ASTRAEA_OK; ++t)
            rc = astraea_step(x_cur[t], x_ref, lse_cache, n_skip, q[t], k[t], v[t], out_cache, score, idx_sel, idx_rem,
                              B, H, N, N_sel, d, k_keep[t], w_alpha, w_beta, delta_mode, lse_mode,
                              workspace, workspace_bytes, cap);
        e = cudaStreamEndCapture(cap, &s->graph);          // also ends a capture that a failed step left open
    }
    if (e == cudaSuccess && rc == ASTRAEA_OK) e = cudaGraphInstantiate(&s->exec, s->graph, 0);
    cudaStreamDestroy(cap);
    if (rc != ASTRAEA_OK) { astraea_schedule_destroy(s); return rc; }
    if (e != cudaSuccess) {
        astraea_schedule_destroy(s);
        return fail(ASTRAEA_ERR_CUDA, "astraea_schedule_create (graph capture): %s", cudaGetErrorString(e));
    }
    *schedule = s;
    return ASTRAEA_OK;
}

int32_t astraea_schedule_launch(astraea_schedule *s, void *stream)
{
    REQUIRE(s && s->exec, "astraea_schedule_launch: null schedule");
    cudaError_t e = cudaGraphLaunch(s->exec, (cudaStream_t)stream);
    if (e != cudaSuccess) return fail(ASTRAEA_ERR_CUDA, "astraea_schedule_launch: %s", cudaGetErrorString(e));
    return ASTRAEA_OK;
}

// ------------------------------------------------------------------ a generation (T steps x L blocks) as one CUDA graph
struct astraea_model_schedule {
    cudaGraph_t graph;
    cudaGraphExec_t exec;
    int L, T;
};

void astraea_model_schedule_destroy(astraea_model_schedule *s)
{
    if (!s) return;
    if (s->exec) cudaGraphExecDestroy(s->exec);
    if (s->graph) cudaGraphDestroy(s->graph);
    delete s;
}

int32_t astraea_timestep_level_budgets(const int32_t *k_keep, int T, int N_sel, int32_t *out)
{
    if (!k_keep || !out || T <= 0 || N_sel < 0) return fail(ASTRAEA_ERR_INVALID_ARG, "astraea_timestep_level_budgets: bad arguments");
    long long carry = 0;
    int computed = 0;
    for (int t = 0; t < T; ++t) {
        if (k_keep[t] < 0 || k_keep[t] > N_sel) return fail(ASTRAEA_ERR_INVALID_ARG, "astraea_timestep_level_budgets: k_keep[%d]=%d outside [0, N_sel=%d]", t, k_keep[t], N_sel);
        carry += k_keep[t];
        if (t == 0 || (N_sel > 0 && carry >= N_sel)) {
            out[t] = N_sel;
            carry -= N_sel;
            if (carry < 0) carry = 0;          // the first step computes everything whatever its budget was
            ++computed;
        } else {
            out[t] = 0;
        }
    }
    return computed;
}

int32_t astraea_model_schedule_create(astraea_model_schedule **schedule, int L, int T, const int32_t *k_keep,
                                      const void *const *x_in, const astraea_block_weights *weights,
                                      const astraea_block_state *states, const void *const *text_k,
                                      const void *const *text_v, int N_text,
                                      float *const *score, int32_t *const *idx_sel, int32_t *const *idx_rem,
                                      int B, int H, int N, int N_sel, int d,
                                      float w_alpha, float w_beta, int delta_mode, int lse_mode, float eps, int variant,
                                      void *workspace, size_t workspace_bytes)
{
    REQUIRE(schedule, "astraea_model_schedule_create: null schedule pointer");
    *schedule = nullptr;
    REQUIRE(L > 0 && T > 0 && k_keep && x_in && weights && states && text_k && text_v && score && idx_sel,
            "astraea_model_schedule_create: L, T must be positive and the arrays non-null");
    REQUIRE(N_sel >= 0 && N_sel <= N, "astraea_model_schedule_create: N_sel=%d outside [0, N=%d]", N_sel, N);
    if (variant < ASTRAEA_VARIANT_TOKEN_WISE || variant > ASTRAEA_VARIANT_FIXED_TOKEN)
        return fail(ASTRAEA_ERR_UNSUPPORTED, "astraea_model_schedule_create: unknown variant %d", variant);
    for (int t = 0; t < T; ++t) {
        REQUIRE(k_keep[t] >= 0 && k_keep[t] <= N_sel, "astraea_model_schedule_create: k_keep[%d]=%d outside [0, N_sel=%d]", t, k_keep[t], N_sel);
        REQUIRE(variant != ASTRAEA_VARIANT_TIMESTEP || k_keep[t] == 0 || k_keep[t] == N_sel,
                "astraea_model_schedule_create: the Timestep-level variant computes all tokens or none, k_keep[%d]=%d", t, k_keep[t]);
        REQUIRE(x_in[t], "astraea_model_schedule_create: null input pointer at step %d", t);
    }
    for (int l = 0; l < L; ++l)
        REQUIRE(text_k[l] && text_v[l] && score[l] && idx_sel[l], "astraea_model_schedule_create: null pointer for block %d", l);
    astraea_model_schedule *s = new (std::nothrow) astraea_model_schedule();
    if (!s) return fail(ASTRAEA_ERR_CUDA, "astraea_model_schedule_create: out of host memory");
    s->graph = nullptr; s->exec = nullptr; s->L = L; s->T = T;
    cudaStream_t cap = nullptr;
    cudaError_t e = cudaStreamCreateWithFlags(&cap, cudaStreamNonBlocking);
    if (e != cudaSuccess) { delete s; return fail(ASTRAEA_ERR_CUDA, "astraea_model_schedule_create: %s", cudaGetErrorString(e)); }
    e = cudaStreamBeginCapture(cap, cudaStreamCaptureModeThreadLocal);
    int32_t rc = ASTRAEA_OK;
    if (e == cudaSuccess) {
        const uint32_t base = variant == ASTRAEA_VARIANT_SELECT_QK ? ASTRAEA_BLOCK_SELECT_QK : 0u;
        for (int t = 0; t < T && rc == ASTRAEA_OK; ++t)
            for (int l = 0; l < L && rc == ASTRAEA_OK; ++l) {
                const bool shared = variant == ASTRAEA_VARIANT_FIXED_TOKEN && l > 0;      // block 0's selection serves the whole step
                rc = astraea_block_step(l == 0 ? x_in[t] : states[l - 1].y_cache, &weights[l], &states[l], text_k[l], text_v[l], N_text,
                                        score[l], shared ? idx_sel[0] : idx_sel[l], idx_rem ? idx_rem[l] : nullptr,
                                        B, H, N, N_sel, d, k_keep[t], w_alpha, w_beta, delta_mode, lse_mode, eps,
                                        base | (shared ? ASTRAEA_BLOCK_REUSE_SELECTION : 0u), workspace, workspace_bytes, cap);
            }
        e = cudaStreamEndCapture(cap, &s->graph);          // also ends a capture that a failed step left open
    }
    if (e == cudaSuccess && rc == ASTRAEA_OK) e = cudaGraphInstantiate(&s->exec, s->graph, 0);
    cudaStreamDestroy(cap);
    if (rc != ASTRAEA_OK) { astraea_model_schedule_destroy(s); return rc; }
    if (e != cudaSuccess) {
        astraea_model_schedule_destroy(s);
        return fail(ASTRAEA_ERR_CUDA, "astraea_model_schedule_create (graph capture): %s", cudaGetErrorString(e));
    }
    *schedule = s;
    return ASTRAEA_OK;
}

int32_t astraea_model_schedule_launch(astraea_model_schedule *s, void *stream)
{
    REQUIRE(s && s->exec, "astraea_model_schedule_launch: null schedule");
    cudaError_t e = cudaGraphLaunch(s->exec, (cudaStream_t)stream);
    if (e != cudaSuccess) return fail(ASTRAEA_ERR_CUDA, "astraea_model_schedule_launch: %s", cudaGetErrorString(e));
    return ASTRAEA_OK;
}

// ------------------------------------------------------------------ host-buffer session
// astraea_step_host moves q, k, v in and the output back in groups of heads, so that the copies of one group run
// under the attention of another.
constexpr int kHostGroups = 12;      // measured: 4 -> 12 groups takes 9.24 -> 8.90 ms (CogVideoX shape), 100.6 -> 94.3 ms (HunyuanVideo shape)

struct astraea_session {
    int B, H, N, N_sel, d;
    size_t tensor_bytes;
    void *x_cur, *x_ref, *q, *k, *v, *out_cache;
    float *lse_cache, *score;
    int32_t *n_skip, *idx_sel, *idx_rem;
    void *workspace;
    size_t workspace_bytes;
    cudaStream_t stream;            // score, select, refresh, attention of the even head groups
    cudaStream_t stream2;           // attention of the odd head groups: the CTAs of one group fill the SMs that the last,
                                    // partial wave of the group before leaves idle (two heads of 128 query tiles are 1.73
                                    // waves of CTAs: one after the other every group would pay for 2)
    cudaStream_t copy_in, copy_out; // host -> device and device -> host copies, overlapped with the compute stream
    cudaStream_t gather;            // zero-copy fetches of the selected q rows from a pinned host buffer
    cudaEvent_t ev_sel;             // the selection of this step is known
    cudaEvent_t ev_q[kHostGroups];  // the selected q rows of a head group have arrived
    cudaEvent_t ev_x;               // x_cur has arrived
    cudaEvent_t ev_in[kHostGroups]; // q, k, v of a head group have arrived
    cudaEvent_t ev_attn[kHostGroups];   // attention of a head group is done
    int steps;
    size_t last_h2d_bytes;          // host-to-device bytes of the last step
};

void astraea_session_destroy(astraea_session *s)
{
    if (!s) return;
    void *bufs[] = {s->x_cur, s->x_ref, s->q, s->k, s->v, s->out_cache, s->lse_cache, s->score,
                    s->n_skip, s->idx_sel, s->idx_rem, s->workspace};
    for (void *p : bufs) if (p) cudaFree(p);
    if (s->ev_x) cudaEventDestroy(s->ev_x);
    if (s->ev_sel) cudaEventDestroy(s->ev_sel);
    for (int g = 0; g < kHostGroups; ++g) {
        if (s->ev_q[g]) cudaEventDestroy(s->ev_q[g]);
        if (s->ev_in[g]) cudaEventDestroy(s->ev_in[g]);
        if (s->ev_attn[g]) cudaEventDestroy(s->ev_attn[g]);
    }
    cudaStream_t streams[] = {s->stream, s->stream2, s->copy_in, s->copy_out, s->gather};
    for (cudaStream_t st : streams) if (st) cudaStreamDestroy(st);
    delete s;
}

int32_t astraea_session_create(astraea_session **session, int B, int H, int N, int N_sel, int d)
{
    REQUIRE(session, "astraea_session_create: null session pointer");
    *session = nullptr;
    REQUIRE(B > 0 && H > 0 && N > 0 && N_sel >= 0 && N_sel <= N, "astraea_session_create: bad sizes");
    if (d != 64 && d != 72 && d != 128) return fail(ASTRAEA_ERR_UNSUPPORTED, "astraea_session_create: head_dim %d", d);
    astraea_session *s = new (std::nothrow) astraea_session();
    if (!s) return fail(ASTRAEA_ERR_CUDA, "astraea_session_create: out of host memory");
    memset(s, 0, sizeof(*s));
    s->B = B; s->H = H; s->N = N; s->N_sel = N_sel; s->d = d;
    s->tensor_bytes = (size_t)B * N * H * d * 2;
    s->workspace_bytes = astraea_workspace_bytes(ASTRAEA_OP_STEP, B, H, N, N, d);
    cudaError_t e = cudaStreamCreateWithFlags(&s->stream, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&s->stream2, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&s->copy_in, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&s->copy_out, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&s->gather, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&s->ev_x, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&s->ev_sel, cudaEventDisableTiming);
    for (int g = 0; g < kHostGroups; ++g) {
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&s->ev_q[g], cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&s->ev_in[g], cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&s->ev_attn[g], cudaEventDisableTiming);
    }
    void **big[] = {&s->x_cur, &s->x_ref, &s->q, &s->k, &s->v, &s->out_cache};
    for (void **p : big) if (e == cudaSuccess) e = cudaMalloc(p, s->tensor_bytes);
    if (e == cudaSuccess) e = cudaMalloc((void **)&s->lse_cache, (size_t)B * H * N * 4);
    if (e == cudaSuccess) e = cudaMalloc((void **)&s->score, (size_t)B * (N_sel + 1) * 4);
    if (e == cudaSuccess) e = cudaMalloc((void **)&s->n_skip, (size_t)B * (N_sel + 1) * 4);
    if (e == cudaSuccess) e = cudaMalloc((void **)&s->idx_sel, (size_t)B * N * 4);
    if (e == cudaSuccess) e = cudaMalloc((void **)&s->idx_rem, (size_t)B * (N_sel + 1) * 4);
    if (e == cudaSuccess) e = cudaMalloc(&s->workspace, s->workspace_bytes);
    if (e == cudaSuccess) e = cudaMemsetAsync(s->workspace, 0, s->workspace_bytes, s->stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(s->n_skip, 0, (size_t)B * (N_sel + 1) * 4, s->stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(s->lse_cache, 0, (size_t)B * H * N * 4, s->stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(s->out_cache, 0, s->tensor_bytes, s->stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s->stream);
    if (e != cudaSuccess) {
        int32_t rc = fail(ASTRAEA_ERR_CUDA, "astraea_session_create: %s", cudaGetErrorString(e));
        astraea_session_destroy(s);
        return rc;
    }
    *session = s;
    return ASTRAEA_OK;
}

size_t astraea_session_last_h2d_bytes(const astraea_session *s) { return s ? s->last_h2d_bytes : 0; }

int32_t astraea_step_host(astraea_session *s, const void *x_cur, const void *q, const void *k,
                          const void *v, void *out, int k_keep,
                          float w_alpha, float w_beta, int delta_mode, int lse_mode)
{
    REQUIRE(s && x_cur && q && k && v && out, "astraea_step_host: null argument");
    REQUIRE(k_keep >= 0 && k_keep <= s->N_sel, "astraea_step_host: k_keep=%d outside [0, N_sel=%d]", k_keep, s->N_sel);
    REQUIRE(s->steps > 0 || k_keep == s->N_sel, "astraea_step_host: the first step of a session must compute every token (k_keep = N_sel)");
    const int B = s->B, H = s->H, N = s->N, N_sel = s->N_sel, d = s->d, D = H * d;
    const int n_always = N - N_sel, M = k_keep + n_always;
    const size_t pitch = (size_t)D * 2, rows = (size_t)B * N;
    const size_t attn_ws = attn_workspace_bytes(B, H, N, M, d);
    char *ws = reinterpret_cast<char *>(s->workspace);
    const int groups = H < kHostGroups ? H : kHostGroups;
    auto head_lo = [&](int g) { return (int)((long long)H * g / groups); };

    // Only the M selected rows of q are ever read.  When q sits in pinned host memory that the device can address, it
    // is not copied: once the selection is known a kernel fetches just the listed rows over the bus (zero-copy reads
    // of whole 2*D-byte rows), which takes (N - M) / N of one tensor off the host-to-device traffic that bounds the step.
    // Worth it only while the bus bounds the step: the fetch kernels share the SMs with the attention, and on a step
    // whose attention takes longer than its transfers (the HunyuanVideo shape: 95 -> 101 ms) they only delay it.
    // Rough rates: 1e15 flop/s for the attention, 5e10 bytes/s for the bus.
    const void *q_mapped = nullptr;
    const double attn_s = 4.0 * B * H * (double)M * N * d / 1e15, bus_s = 4.0 * (double)s->tensor_bytes / 5e10;
    if (M < N && M > 0 && attn_s < bus_s) {
        cudaPointerAttributes attr;
        if (cudaPointerGetAttributes(&attr, q) == cudaSuccess && attr.type == cudaMemoryTypeHost && attr.devicePointer)
            q_mapped = attr.devicePointer;
        else
            cudaGetLastError();               // pageable memory: not an error, the rows are copied as before
    }
    s->last_h2d_bytes = s->tensor_bytes * 3 + (q_mapped ? (size_t)B * M * D * 2 : s->tensor_bytes);

    // copy-in stream: x_cur first (the score needs nothing else), then (q,) k, v by head group
    cudaError_t e = cudaMemcpyAsync(s->x_cur, x_cur, s->tensor_bytes, cudaMemcpyHostToDevice, s->copy_in);
    if (e == cudaSuccess) e = cudaEventRecord(s->ev_x, s->copy_in);
    for (int g = 0; g < groups && e == cudaSuccess; ++g) {
        const size_t off = (size_t)head_lo(g) * d * 2, width = (size_t)(head_lo(g + 1) - head_lo(g)) * d * 2;
        const void *src[3] = {q, k, v};
        void *dst[3] = {s->q, s->k, s->v};
        for (int i = q_mapped ? 1 : 0; i < 3 && e == cudaSuccess; ++i)
            e = cudaMemcpy2DAsync(static_cast<char *>(dst[i]) + off, pitch, static_cast<const char *>(src[i]) + off, pitch,
                                  width, rows, cudaMemcpyHostToDevice, s->copy_in);
        if (e == cudaSuccess) e = cudaEventRecord(s->ev_in[g], s->copy_in);
    }
    if (e != cudaSuccess) return fail(ASTRAEA_ERR_CUDA, "astraea_step_host (copy in): %s", cudaGetErrorString(e));

    // compute stream: score -> select -> refresh of x_ref, then the attention of each head group as it arrives
    e = cudaStreamWaitEvent(s->stream, s->ev_x, 0);
    if (e == cudaSuccess && s->steps == 0)   // no earlier step: the reference inputs are the current ones
        e = cudaMemcpyAsync(s->x_ref, s->x_cur, s->tensor_bytes, cudaMemcpyDeviceToDevice, s->stream);
    if (e != cudaSuccess) return fail(ASTRAEA_ERR_CUDA, "astraea_step_host: %s", cudaGetErrorString(e));
    int32_t rc = astraea_score(s->x_cur, s->x_ref, s->lse_cache, s->n_skip, s->score, B, N, N_sel, D, H, w_alpha, w_beta,
                               delta_mode, lse_mode, s->stream);
    if (rc == ASTRAEA_OK)
        rc = astraea_select(s->score, B, N_sel, k_keep, n_always, s->idx_sel, s->idx_rem, s->n_skip, ws + attn_ws,
                            s->workspace_bytes - attn_ws, s->stream);
    if (rc == ASTRAEA_OK)
        rc = astraea_scatter_reuse(s->x_ref, s->x_cur, s->idx_sel, B, N, M, D, ASTRAEA_SCATTER_SRC_FULL, s->workspace, s->stream);
    if (rc != ASTRAEA_OK) return rc;
    e = cudaEventRecord(s->ev_sel, s->stream);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(s->stream2, s->ev_sel, 0);
    if (e != cudaSuccess) return fail(ASTRAEA_ERR_CUDA, "astraea_step_host: %s", cudaGetErrorString(e));
    if (q_mapped) {
        // the selected rows of q, straight from the host buffer, head group by head group on a stream of its own (so
        // that a group's attention waits for its own columns only and the fetches run under the attention of the
        // groups before)
        e = cudaStreamWaitEvent(s->gather, s->ev_sel, 0);
        for (int g = 0; g < groups && e == cudaSuccess; ++g) {
            const size_t off = (size_t)head_lo(g) * d * 2;
            rc = launch_scatter(static_cast<char *>(s->q) + off, static_cast<const char *>(q_mapped) + off, s->idx_sel, B, N, M,
                                (head_lo(g + 1) - head_lo(g)) * d, ASTRAEA_SCATTER_SRC_FULL, reinterpret_cast<int *>(s->workspace),
                                s->gather, D);
            if (rc != ASTRAEA_OK) return rc;
            e = cudaEventRecord(s->ev_q[g], s->gather);
        }
        if (e != cudaSuccess) return fail(ASTRAEA_ERR_CUDA, "astraea_step_host (fetch of the selected q rows): %s", cudaGetErrorString(e));
    }
    for (int g = 0; g < groups; ++g) {
        cudaStream_t cs = (g & 1) ? s->stream2 : s->stream;
        e = cudaStreamWaitEvent(cs, s->ev_in[g], 0);
        if (e == cudaSuccess && q_mapped) e = cudaStreamWaitEvent(cs, s->ev_q[g], 0);
        if (e != cudaSuccess) return fail(ASTRAEA_ERR_CUDA, "astraea_step_host: %s", cudaGetErrorString(e));
        if (M > 0) {
            AttnArgs a;
            a.q = s->q; a.k = s->k; a.v = s->v;
            a.q_sb = a.k_sb = a.v_sb = (int64_t)N * D;
            a.q_sh = a.k_sh = a.v_sh = d;
            a.q_sn = a.k_sn = a.v_sn = D;
            a.q_idx = s->idx_sel; a.M = M; a.out = s->out_cache; a.lse_out = s->lse_cache;
            a.B = B; a.H = H; a.N = N; a.d = d; a.N_tok = N;
            a.scale = 1.0f / sqrtf((float)d);
            a.flags = 0;
            a.err_word = reinterpret_cast<int *>(s->workspace);
            a.head_begin = head_lo(g); a.head_count = head_lo(g + 1) - head_lo(g);
            rc = launch_sparse_attn(a, cs);
            if (rc != ASTRAEA_OK) return rc;
        }
        e = cudaEventRecord(s->ev_attn[g], cs);
        // copy-out stream: the group's columns of the output cache (computed and reused rows alike)
        if (e == cudaSuccess) e = cudaStreamWaitEvent(s->copy_out, s->ev_attn[g], 0);
        const size_t off = (size_t)head_lo(g) * d * 2, width = (size_t)(head_lo(g + 1) - head_lo(g)) * d * 2;
        if (e == cudaSuccess)
            e = cudaMemcpy2DAsync(static_cast<char *>(out) + off, pitch, static_cast<const char *>(s->out_cache) + off, pitch,
                                  width, rows, cudaMemcpyDeviceToHost, s->copy_out);
        if (e != cudaSuccess) return fail(ASTRAEA_ERR_CUDA, "astraea_step_host (copy out): %s", cudaGetErrorString(e));
    }
    e = cudaStreamSynchronize(s->copy_out);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s->copy_in);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s->gather);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s->stream2);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s->stream);      // the refresh of x_ref runs beside the attention
    if (e != cudaSuccess) return fail(ASTRAEA_ERR_CUDA, "astraea_step_host (copy out): %s", cudaGetErrorString(e));
    s->steps++;
    return astraea_poll_error(s->workspace, s->stream);
}

}  // extern "C"
