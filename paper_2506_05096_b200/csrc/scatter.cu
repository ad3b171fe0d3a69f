// astraea_scatter_reuse: cache[b, idx[b,r], :] = rows[b, r, :] (or rows[b, idx[b,r], :]);
// rows that are not listed keep the cached value of the earlier step (Algorithm 1 lines 6-7).
//
// HBM-bound row copy: one warp per row, 16-byte vectors, several loads in flight per lane,
// grid a multiple of the SM count with a grid stride over the rows.
#include "common.cuh"

namespace astraea {
namespace {

constexpr int kWarpsPerBlock = 8;
constexpr int kBlocksPerSM = 16;
constexpr int kUnroll = 6;

__device__ __forceinline__ uint4 ld_stream(const uint4 *p) {
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
    return r;
}

__global__ void __launch_bounds__(kWarpsPerBlock * 32)
scatter_kernel(uint4 *__restrict__ cache, const uint4 *__restrict__ rows, const int32_t *__restrict__ idx,
               int B, int N, int M, int vec_per_row, int src_full, int *__restrict__ err_word)
{
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const long long total = (long long)B * M;
    for (long long t = (long long)blockIdx.x * kWarpsPerBlock + warp; t < total;
         t += (long long)gridDim.x * kWarpsPerBlock) {
        const int b = (int)(t / M);
        const int r = (int)(t - (long long)b * M);
        const int i = __ldg(idx + t);
        // never write outside the cache, and never write a row twice: an entry that is out of range or does not
        // exceed its predecessor is skipped and reported
        if ((unsigned)i >= (unsigned)N || (r > 0 && __ldg(idx + t - 1) >= i)) {
            if (lane == 0 && err_word) atomicExch(err_word, kErrBadIndex);
            continue;
        }
        const uint4 *src = rows + ((size_t)b * (src_full ? N : M) + (src_full ? i : r)) * vec_per_row;
        uint4 *dst = cache + ((size_t)b * N + i) * vec_per_row;
        for (int v = lane; v < vec_per_row; v += 32 * kUnroll) {
            uint4 a[kUnroll];
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) if (v + 32 * u < vec_per_row) a[u] = ld_stream(src + v + 32 * u);
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) if (v + 32 * u < vec_per_row) dst[v + 32 * u] = a[u];
        }
    }
}

}  // namespace

int32_t launch_scatter(void *cache, const void *rows, const int32_t *idx, int B, int N, int M,
                       int row_elems, uint32_t flags, int *err_word, cudaStream_t stream)
{
    const long long total = (long long)B * M;
    if (total == 0) return ASTRAEA_OK;
    long long want = (total + kWarpsPerBlock - 1) / kWarpsPerBlock;
    const long long cap = (long long)sm_count() * kBlocksPerSM;
    int grid = (int)(want < cap ? want : cap);
    scatter_kernel<<<grid, kWarpsPerBlock * 32, 0, stream>>>(
        reinterpret_cast<uint4 *>(cache), reinterpret_cast<const uint4 *>(rows), idx, B, N, M,
        row_elems >> 3, (flags & ASTRAEA_SCATTER_SRC_FULL) ? 1 : 0, err_word);
    return check_launch("astraea_scatter_reuse");
}

}  // namespace astraea
