// astraea_score: S_token = w_alpha * S_LSE * Delta_token + w_beta * e^{n}
// (selection-metric equations of Section 3.2; Algorithm 1 lines 1-2).
//
// HBM-bound: 2 * D bf16 per token are read once.  One warp (half or a quarter of one for narrow
// rows) owns one token row and streams it with 16-byte loads, six per tensor in flight per lane; the
// channel reduction is a per-lane fp32 partial sum followed by a shuffle tree.  The per-head LSE values of
// the token (a strided gather of H floats, 1/d of the traffic) are averaged by the same
// warp.  The grid is a multiple of the SM count and walks the tokens with a grid stride.
#include "common.cuh"

namespace astraea {
namespace {

constexpr int kWarpsPerBlock = 8;
constexpr int kBlocksPerSM = 16;     // twice what is resident: the second half evens out the tail
constexpr int kUnroll = 6;           // 16-byte loads in flight per lane and tensor

__device__ __forceinline__ uint4 ld_stream(const uint4 *p) {
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
    return r;
}

template <int MODE>
__device__ __forceinline__ float accum_pair(uint32_t a, uint32_t b, float acc) {
    // two bf16 per word: low half = even element
    float a0 = __uint_as_float(a << 16), a1 = __uint_as_float(a & 0xffff0000u);
    float b0 = __uint_as_float(b << 16), b1 = __uint_as_float(b & 0xffff0000u);
    float d0 = a0 - b0, d1 = a1 - b1;
    if (MODE == ASTRAEA_DELTA_MEAN_ABS) return acc + fabsf(d0) + fabsf(d1);
    if (MODE == ASTRAEA_DELTA_MEAN_SQ) return fmaf(d1, d1, fmaf(d0, d0, acc));
    return acc + d0 + d1;
}

template <int MODE>
__device__ __forceinline__ float accum_vec(const uint4 &a, const uint4 &b, float acc) {
    acc = accum_pair<MODE>(a.x, b.x, acc);
    acc = accum_pair<MODE>(a.y, b.y, acc);
    acc = accum_pair<MODE>(a.z, b.z, acc);
    acc = accum_pair<MODE>(a.w, b.w, acc);
    return acc;
}

// LPR lanes share one token row: 32 for rows of 64 or more 16-byte vectors; 16 or 8 for narrower ones, so that no lane
// of a warp is left without loads.  (Splitting the 144-vector rows of the Open-Sora shape over half-warps was
// measured and is slower than a whole warp per row, 33.8 against 31.8 us: what bounds the kernel there is its fixed
// launch / ramp / tail time of ~5 us on 25 us of streaming, not the load slots.)
template <int MODE, int LPR>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
score_kernel(const uint4 *__restrict__ x_cur, const uint4 *__restrict__ x_ref,
             const float *__restrict__ lse, const int32_t *__restrict__ n_skip,
             float *__restrict__ score, int B, int N, int N_sel, int D, int H,
             float w_alpha, float w_beta, int lse_mode, float *__restrict__ part)
{
    // a kernel launched behind this one with programmatic stream serialization (the selection) may become resident
    // and set itself up as soon as SMs free up; it still waits for this whole grid before it reads the scores
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    constexpr int kRowsPerWarp = 32 / LPR;
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int sub = lane / LPR, sl = lane % LPR;          // which of the warp's rows, and the lane within that row
    const int vec_per_row = D >> 3;                       // 16-byte vectors per row
    const long long total = (long long)B * N_sel;
    const float inv_D = 1.0f / (float)D;
    const float inv_H = 1.0f / (float)H;

    for (long long t0 = ((long long)blockIdx.x * kWarpsPerBlock + warp) * kRowsPerWarp; t0 < total;
         t0 += (long long)gridDim.x * kWarpsPerBlock * kRowsPerWarp) {
        const long long t = t0 + sub;
        const bool have = t < total;
        const int b = have ? (int)(t / N_sel) : 0;
        const int i = have ? (int)(t - (long long)b * N_sel) : 0;
        const size_t row = ((size_t)b * N + i) * vec_per_row;
        const uint4 *pc = x_cur + row;
        const uint4 *pr = x_ref + row;

        // the token's per-head LSE values (a strided gather of H floats) and its counter are requested BEFORE the row
        // is streamed, so that their latency runs under the row's loads instead of after them (with the gather behind
        // the row loop every row cost two memory round trips and the kernel streamed 14 % below what the loads alone do)
        constexpr int kLsePre = 2;                       // heads per lane that are prefetched: H <= 2 * LPR
        float lv[kLsePre];
#pragma unroll
        for (int u = 0; u < kLsePre; ++u) {
            const int h = sl + LPR * u;
            lv[u] = (lse != nullptr && have && h < H) ? __ldg(lse + ((size_t)b * H + h) * N + i) : 0.f;
        }
        int n = (n_skip != nullptr && have && sl == 0) ? n_skip[(size_t)b * N_sel + i] : 0;

        float acc0 = 0.f, acc1 = 0.f;
        for (int v = sl; have && v < vec_per_row; v += LPR * kUnroll) {
            uint4 a[kUnroll], r[kUnroll];
            // loads past the end of the row are skipped; zeros add nothing in any of the three reductions
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) a[u] = (v + LPR * u < vec_per_row) ? ld_stream(pc + v + LPR * u) : make_uint4(0, 0, 0, 0);
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) r[u] = (v + LPR * u < vec_per_row) ? ld_stream(pr + v + LPR * u) : make_uint4(0, 0, 0, 0);
#pragma unroll
            for (int u = 0; u < kUnroll; u += 2) {
                acc0 = accum_vec<MODE>(a[u], r[u], acc0);
                acc1 = accum_vec<MODE>(a[u + 1], r[u + 1], acc1);
            }
        }
        float acc = acc0 + acc1;

        // S_LSE: mean over heads of exp(lse[b,h,i]) (or of lse itself); the log value is clamped like the skip
        // counters so that the exponential stays finite in fp32
        float ls = 0.f;
        if (lse != nullptr && have) {
#pragma unroll
            for (int u = 0; u < kLsePre; ++u)
                if (sl + LPR * u < H) ls += (lse_mode == ASTRAEA_LSE_SUM_EXP) ? expf(fminf(lv[u], (float)ASTRAEA_LSE_CLAMP)) : lv[u];
            for (int h = sl + LPR * kLsePre; h < H; h += LPR) {          // more than 2 * LPR heads: the rest afterwards
                float l = __ldg(lse + ((size_t)b * H + h) * N + i);
                ls += (lse_mode == ASTRAEA_LSE_SUM_EXP) ? expf(fminf(l, (float)ASTRAEA_LSE_CLAMP)) : l;
            }
        }
#pragma unroll
        for (int o = LPR / 2; o > 0; o >>= 1) {
            acc += __shfl_xor_sync(0xffffffffu, acc, o);
            ls += __shfl_xor_sync(0xffffffffu, ls, o);
        }
        if (sl == 0 && have && part != nullptr) {
            // a shard of the channels / heads: the raw sums, to be added up over the shards before they are combined
            part[(size_t)b * N_sel + i] = acc;
            part[((size_t)B + b) * N_sel + i] = ls;
        } else if (sl == 0 && have) {
            float delta = acc * inv_D;
            float s_lse = (lse != nullptr) ? ls * inv_H : 1.0f;
            n = min(n, ASTRAEA_N_SKIP_CLAMP);
            score[(size_t)b * N_sel + i] = w_alpha * (s_lse * delta) + w_beta * expf((float)n);
        }
    }
}

template <int MODE>
void launch_mode(int lpr, int grid, cudaStream_t stream, const uint4 *xc, const uint4 *xr, const float *lse, const int32_t *n_skip,
                 float *score, int B, int N, int N_sel, int D, int H, float w_alpha, float w_beta, int lse_mode, float *part)
{
    dim3 block(kWarpsPerBlock * 32);
    if (lpr == 32) score_kernel<MODE, 32><<<grid, block, 0, stream>>>(xc, xr, lse, n_skip, score, B, N, N_sel, D, H, w_alpha, w_beta, lse_mode, part);
    else if (lpr == 16) score_kernel<MODE, 16><<<grid, block, 0, stream>>>(xc, xr, lse, n_skip, score, B, N, N_sel, D, H, w_alpha, w_beta, lse_mode, part);
    else score_kernel<MODE, 8><<<grid, block, 0, stream>>>(xc, xr, lse, n_skip, score, B, N, N_sel, D, H, w_alpha, w_beta, lse_mode, part);
}

// score[b, i] = w_alpha * (sum of exp(lse) / H) * (sum of differences / D) + w_beta * e^n from the summed partial sums
__global__ void __launch_bounds__(256)
score_combine_kernel(const float *__restrict__ part, const int32_t *__restrict__ n_skip, float *__restrict__ score,
                     long long total, float inv_D, float inv_H, int has_lse, float w_alpha, float w_beta)
{
    for (long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x; t < total; t += (long long)gridDim.x * blockDim.x) {
        const float delta = part[t] * inv_D;
        const float s_lse = has_lse ? part[total + t] * inv_H : 1.0f;
        int n = n_skip ? n_skip[t] : 0;
        n = min(n, ASTRAEA_N_SKIP_CLAMP);
        score[t] = w_alpha * (s_lse * delta) + w_beta * expf((float)n);
    }
}

}  // namespace

int32_t launch_score_combine(const float *part, const int32_t *n_skip, float *score, int B, int N_sel, int D, int H,
                             int has_lse, float w_alpha, float w_beta, cudaStream_t stream)
{
    const long long total = (long long)B * N_sel;
    if (total == 0) return ASTRAEA_OK;
    const long long want = (total + 255) / 256, cap = (long long)sm_count() * 8;
    score_combine_kernel<<<(int)(want < cap ? want : cap), 256, 0, stream>>>(part, n_skip, score, total, 1.0f / (float)D, 1.0f / (float)H,
                                                                             has_lse, w_alpha, w_beta);
    return check_launch("astraea_score_combine");
}

int32_t launch_score(const void *x_cur, const void *x_ref, const float *lse, const int32_t *n_skip,
                     float *score, int B, int N, int N_sel, int D, int H, float w_alpha, float w_beta,
                     int delta_mode, int lse_mode, cudaStream_t stream, float *part)
{
    const long long total = (long long)B * N_sel;
    if (total == 0) return ASTRAEA_OK;
    const int vec_per_row = D >> 3;
    const int lpr = vec_per_row >= 64 ? 32 : vec_per_row >= 32 ? 16 : 8;     // lanes per row: every lane gets at least two vectors
    const long long rows_per_block = (long long)kWarpsPerBlock * (32 / lpr);
    long long want = (total + rows_per_block - 1) / rows_per_block;
    const long long cap = (long long)sm_count() * kBlocksPerSM;
    int grid = (int)(want < cap ? want : cap);
    const uint4 *xc = reinterpret_cast<const uint4 *>(x_cur);
    const uint4 *xr = reinterpret_cast<const uint4 *>(x_ref);
    switch (delta_mode) {
    case ASTRAEA_DELTA_MEAN_ABS:
        launch_mode<ASTRAEA_DELTA_MEAN_ABS>(lpr, grid, stream, xc, xr, lse, n_skip, score, B, N, N_sel, D, H, w_alpha, w_beta, lse_mode, part);
        break;
    case ASTRAEA_DELTA_MEAN_SQ:
        launch_mode<ASTRAEA_DELTA_MEAN_SQ>(lpr, grid, stream, xc, xr, lse, n_skip, score, B, N, N_sel, D, H, w_alpha, w_beta, lse_mode, part);
        break;
    default:
        launch_mode<ASTRAEA_DELTA_MEAN_SIGNED>(lpr, grid, stream, xc, xr, lse, n_skip, score, B, N, N_sel, D, H, w_alpha, w_beta, lse_mode, part);
        break;
    }
    return check_launch("astraea_score");
}

}  // namespace astraea
