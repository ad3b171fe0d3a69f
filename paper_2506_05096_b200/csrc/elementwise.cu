// astraea_layernorm_modulate: y[r, :] = LayerNorm(x[r, :]) * (1 + scale[b, :]) + shift[b, :] for the listed token rows
// (Section 3.2: the layers of a compute block other than self-attention act on every token by itself, so the
// element-wise step in front of them runs for the selected tokens only; in front of the key / value projections it
// runs for all tokens).
//
// HBM-bound: every row is read once and written once.  One warp owns one row and keeps it packed in registers (16-byte
// loads, all in flight at once), takes mean and variance from the registers in one pass over shifted data, then
// normalises, modulates and stores in a second pass over the registers.  fp32 arithmetic, one rounding to bf16 at the end.
#include "common.cuh"

namespace astraea {
namespace {

constexpr int kWarpsPerBlock = 8;
constexpr int kBlocksPerSM = 8;
constexpr int kMaxVecPerLane = 16;     // rows of up to 32 * 16 * 8 = 4096 channels

__device__ __forceinline__ uint4 ld_stream(const uint4 *p) {
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
    return r;
}
__device__ __forceinline__ void unpack8(const uint4 &v, float (&f)[8]) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) { f[2 * i] = __uint_as_float(w[i] << 16); f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u); }
}

// VPL: 16-byte vectors per lane (compile-time bound of the register array; vec_per_row <= 32 * VPL)
// (two or three blocks per SM: the row stays packed in registers and is unpacked again in every pass, instead of being
// kept as 8 * VPL floats, which would leave room for one block per SM only and too few bytes in flight)
template <int VPL>
__global__ void __launch_bounds__(kWarpsPerBlock * 32, VPL <= 8 ? 3 : 2)
layernorm_modulate_kernel(const uint4 *__restrict__ x, const int32_t *__restrict__ idx, int M, const uint4 *__restrict__ scale,
                          const uint4 *__restrict__ shift, uint4 *__restrict__ y, int B, int N, int vec_per_row, float eps,
                          int compact_in, int compact_out, int *__restrict__ err_word)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const long long total = (long long)B * M;
    const float inv_D = 1.0f / (float)(vec_per_row * 8);
    for (long long t = (long long)blockIdx.x * kWarpsPerBlock + warp; t < total; t += (long long)gridDim.x * kWarpsPerBlock) {
        const int b = (int)(t / M), r = (int)(t - (long long)b * M);
        const int tok = idx ? __ldg(idx + t) : r;
        if ((unsigned)tok >= (unsigned)N || (idx && r > 0 && __ldg(idx + t - 1) >= tok)) {      // see astraea_scatter_reuse
            if (lane == 0 && err_word) atomicExch(err_word, kErrBadIndex);
            continue;
        }
        const uint4 *src = x + (compact_in ? t : (long long)b * N + tok) * vec_per_row;
        uint4 *dst = y + (compact_out ? t : (long long)b * N + tok) * vec_per_row;
        uint4 v[VPL];
#pragma unroll
        for (int u = 0; u < VPL; ++u) v[u] = (lane + 32 * u < vec_per_row) ? ld_stream(src + lane + 32 * u) : make_uint4(0, 0, 0, 0);
        // mean and variance in one pass over the packed registers, on data shifted by the row's first element: the
        // shift takes the cancellation out of E[(x - x0)^2] - (E[x - x0])^2 whenever the mean is large against the spread
        const float x0 = __shfl_sync(0xffffffffu, __uint_as_float(v[0].x << 16), 0);
        float s1 = 0.f, s2 = 0.f;
#pragma unroll
        for (int u = 0; u < VPL; ++u) {
            if (lane + 32 * u < vec_per_row) {
                float f[8];
                unpack8(v[u], f);
#pragma unroll
                for (int i = 0; i < 8; ++i) { const float c = f[i] - x0; s1 += c; s2 = fmaf(c, c, s2); }
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) { s1 += __shfl_xor_sync(0xffffffffu, s1, o); s2 += __shfl_xor_sync(0xffffffffu, s2, o); }
        const float ms = s1 * inv_D, mean = x0 + ms;
        const float sq = fmaxf(s2 - s1 * ms, 0.f);                 // sum of squares about the mean
        const float rstd = rsqrtf(sq * inv_D + eps);
#pragma unroll
        for (int u = 0; u < VPL; ++u) {
            const int c = lane + 32 * u;
            if (c < vec_per_row) {
                float f[8], sc[8], sh[8];
                unpack8(v[u], f);
                if (scale) unpack8(__ldg(scale + (long long)b * vec_per_row + c), sc);
                if (shift) unpack8(__ldg(shift + (long long)b * vec_per_row + c), sh);
                uint32_t w[4];
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    f[i] = (f[i] - mean) * rstd;
                    if (scale) f[i] = fmaf(f[i], sc[i], f[i]);
                    if (shift) f[i] += sh[i];
                }
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    __nv_bfloat162 v2 = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
                    w[i] = *reinterpret_cast<uint32_t *>(&v2);
                }
                dst[c] = make_uint4(w[0], w[1], w[2], w[3]);
            }
        }
    }
}

}  // namespace

int32_t launch_layernorm_modulate(const void *x, const int32_t *idx, int M, const void *scale, const void *shift, void *y,
                                  int B, int N, int D, float eps, uint32_t flags, int *err_word, cudaStream_t stream)
{
    const int rows = idx ? M : N;
    const long long total = (long long)B * rows;
    if (total == 0) return ASTRAEA_OK;
    const int vec_per_row = D >> 3;
    if (vec_per_row > 32 * kMaxVecPerLane)
        return fail(ASTRAEA_ERR_UNSUPPORTED, "astraea_layernorm_modulate: D=%d above %d", D, 32 * kMaxVecPerLane * 8);
    long long want = (total + kWarpsPerBlock - 1) / kWarpsPerBlock;
    const long long cap = (long long)sm_count() * kBlocksPerSM;
    const int grid = (int)(want < cap ? want : cap);
    const uint4 *xs = reinterpret_cast<const uint4 *>(x), *sc = reinterpret_cast<const uint4 *>(scale), *sh = reinterpret_cast<const uint4 *>(shift);
    uint4 *ys = reinterpret_cast<uint4 *>(y);
    const int ci = (flags & ASTRAEA_LN_COMPACT_IN) ? 1 : 0, co = (flags & ASTRAEA_LN_COMPACT_OUT) ? 1 : 0;
    dim3 block(kWarpsPerBlock * 32);
    if (vec_per_row <= 32 * 4)
        layernorm_modulate_kernel<4><<<grid, block, 0, stream>>>(xs, idx, rows, sc, sh, ys, B, N, vec_per_row, eps, ci, co, err_word);
    else if (vec_per_row <= 32 * 8)
        layernorm_modulate_kernel<8><<<grid, block, 0, stream>>>(xs, idx, rows, sc, sh, ys, B, N, vec_per_row, eps, ci, co, err_word);
    else if (vec_per_row <= 32 * 12)
        layernorm_modulate_kernel<12><<<grid, block, 0, stream>>>(xs, idx, rows, sc, sh, ys, B, N, vec_per_row, eps, ci, co, err_word);
    else
        layernorm_modulate_kernel<16><<<grid, block, 0, stream>>>(xs, idx, rows, sc, sh, ys, B, N, vec_per_row, eps, ci, co, err_word);
    return check_launch("astraea_layernorm_modulate");
}

}  // namespace astraea
