// astraea_score: S_token = w_alpha * S_LSE * Delta_token + w_beta * e^{n}
// (selection-metric equations of Section 3.2; Algorithm 1 lines 1-2).
//
// HBM-bound: 2 * D bf16 per token are read once.  One warp owns one token row and
// streams it with 16-byte loads, six per tensor in flight per lane; the channel reduction is a
// per-lane fp32 partial sum followed by a warp shuffle tree.  The per-head LSE values of
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

template <int MODE>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
score_kernel(const uint4 *__restrict__ x_cur, const uint4 *__restrict__ x_ref,
             const float *__restrict__ lse, const int32_t *__restrict__ n_skip,
             float *__restrict__ score, int B, int N, int N_sel, int D, int H,
             float w_alpha, float w_beta, int lse_mode)
{
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int vec_per_row = D >> 3;                       // 16-byte vectors per row
    const long long total = (long long)B * N_sel;
    const float inv_D = 1.0f / (float)D;
    const float inv_H = 1.0f / (float)H;

    for (long long t = (long long)blockIdx.x * kWarpsPerBlock + warp; t < total;
         t += (long long)gridDim.x * kWarpsPerBlock) {
        const int b = (int)(t / N_sel);
        const int i = (int)(t - (long long)b * N_sel);
        const size_t row = ((size_t)b * N + i) * vec_per_row;
        const uint4 *pc = x_cur + row;
        const uint4 *pr = x_ref + row;

        float acc0 = 0.f, acc1 = 0.f;
        for (int v = lane; v < vec_per_row; v += 32 * kUnroll) {
            uint4 a[kUnroll], r[kUnroll];
            // loads past the end of the row are skipped; zeros add nothing in any of the three reductions
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) a[u] = (v + 32 * u < vec_per_row) ? ld_stream(pc + v + 32 * u) : make_uint4(0, 0, 0, 0);
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) r[u] = (v + 32 * u < vec_per_row) ? ld_stream(pr + v + 32 * u) : make_uint4(0, 0, 0, 0);
#pragma unroll
            for (int u = 0; u < kUnroll; u += 2) {
                acc0 = accum_vec<MODE>(a[u], r[u], acc0);
                acc1 = accum_vec<MODE>(a[u + 1], r[u + 1], acc1);
            }
        }
        float acc = acc0 + acc1;

        // S_LSE: mean over heads of exp(lse[b,h,i]) (or of lse itself)
        float ls = 0.f;
        if (lse != nullptr) {
            for (int h = lane; h < H; h += 32) {
                float l = __ldg(lse + ((size_t)b * H + h) * N + i);
                ls += (lse_mode == ASTRAEA_LSE_SUM_EXP) ? expf(l) : l;
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            acc += __shfl_xor_sync(0xffffffffu, acc, o);
            ls += __shfl_xor_sync(0xffffffffu, ls, o);
        }
        if (lane == 0) {
            float delta = acc * inv_D;
            float s_lse = (lse != nullptr) ? ls * inv_H : 1.0f;
            int n = (n_skip != nullptr) ? n_skip[(size_t)b * N_sel + i] : 0;
            n = min(n, ASTRAEA_N_SKIP_CLAMP);
            score[(size_t)b * N_sel + i] = w_alpha * (s_lse * delta) + w_beta * expf((float)n);
        }
    }
}

}  // namespace

int32_t launch_score(const void *x_cur, const void *x_ref, const float *lse, const int32_t *n_skip,
                     float *score, int B, int N, int N_sel, int D, int H, float w_alpha, float w_beta,
                     int delta_mode, int lse_mode, cudaStream_t stream)
{
    const long long total = (long long)B * N_sel;
    if (total == 0) return ASTRAEA_OK;
    long long want = (total + kWarpsPerBlock - 1) / kWarpsPerBlock;
    const long long cap = (long long)sm_count() * kBlocksPerSM;
    int grid = (int)(want < cap ? want : cap);
    const uint4 *xc = reinterpret_cast<const uint4 *>(x_cur);
    const uint4 *xr = reinterpret_cast<const uint4 *>(x_ref);
    dim3 block(kWarpsPerBlock * 32);
    switch (delta_mode) {
    case ASTRAEA_DELTA_MEAN_ABS:
        score_kernel<ASTRAEA_DELTA_MEAN_ABS><<<grid, block, 0, stream>>>(xc, xr, lse, n_skip, score, B, N, N_sel, D, H, w_alpha, w_beta, lse_mode);
        break;
    case ASTRAEA_DELTA_MEAN_SQ:
        score_kernel<ASTRAEA_DELTA_MEAN_SQ><<<grid, block, 0, stream>>>(xc, xr, lse, n_skip, score, B, N, N_sel, D, H, w_alpha, w_beta, lse_mode);
        break;
    default:
        score_kernel<ASTRAEA_DELTA_MEAN_SIGNED><<<grid, block, 0, stream>>>(xc, xr, lse, n_skip, score, B, N, N_sel, D, H, w_alpha, w_beta, lse_mode);
        break;
    }
    return check_launch("astraea_score");
}

}  // namespace astraea
