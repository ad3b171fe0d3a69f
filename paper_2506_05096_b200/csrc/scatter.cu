// astraea_scatter_reuse: cache[b, idx[b,r], :] = rows[b, r, :] (or rows[b, idx[b,r], :]);
// rows that are not listed keep the cached value of the earlier step (Algorithm 1 lines 6-7).
//
// HBM-bound row copy: one warp (half or a quarter of one for narrow rows) per row, 16-byte vectors,
// several loads in flight per lane, grid a multiple of the SM count with a grid stride over the rows.
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

// LPR lanes copy one row: 32 for wide rows; 16 or 8 for narrow ones, so that a warp moves two or four rows at once and
// every lane keeps several 16-byte loads in flight.
template <int LPR>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
scatter_kernel(uint4 *__restrict__ cache, const uint4 *__restrict__ rows, const int32_t *__restrict__ idx,
               int B, int N, int M, int vec_per_row, int pitch_vec, int src_full, int *__restrict__ err_word)
{
    // vec_per_row 16-byte vectors are copied per row; rows are pitch_vec vectors apart in both tensors (a column slice
    // of wider rows when pitch_vec > vec_per_row: the caller offsets the base pointers to the slice's first column)
    constexpr int kRowsPerWarp = 32 / LPR;
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int sub = lane / LPR, sl = lane % LPR;
    const long long total = (long long)B * M;
    for (long long t0 = ((long long)blockIdx.x * kWarpsPerBlock + warp) * kRowsPerWarp; t0 < total;
         t0 += (long long)gridDim.x * kWarpsPerBlock * kRowsPerWarp) {
        const long long t = t0 + sub;
        if (t >= total) continue;
        const int b = (int)(t / M);
        const int r = (int)(t - (long long)b * M);
        const int i = __ldg(idx + t);
        // never write outside the cache, and never write a row twice: an entry that is out of range or does not
        // exceed its predecessor is skipped and reported
        if ((unsigned)i >= (unsigned)N || (r > 0 && __ldg(idx + t - 1) >= i)) {
            if (sl == 0 && err_word) atomicExch(err_word, kErrBadIndex);
            continue;
        }
        const uint4 *src = rows + ((size_t)b * (src_full ? N : M) + (src_full ? i : r)) * pitch_vec;
        uint4 *dst = cache + ((size_t)b * N + i) * pitch_vec;
        for (int v = sl; v < vec_per_row; v += LPR * kUnroll) {
            uint4 a[kUnroll];
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) if (v + LPR * u < vec_per_row) a[u] = ld_stream(src + v + LPR * u);
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) if (v + LPR * u < vec_per_row) dst[v + LPR * u] = a[u];
        }
    }
}

}  // namespace

int32_t launch_scatter(void *cache, const void *rows, const int32_t *idx, int B, int N, int M,
                       int row_elems, uint32_t flags, int *err_word, cudaStream_t stream, int pitch_elems)
{
    const int pitch_vec = (pitch_elems > 0 ? pitch_elems : row_elems) >> 3;
    const long long total = (long long)B * M;
    if (total == 0) return ASTRAEA_OK;
    const int vec_per_row = row_elems >> 3;
    const int lpr = vec_per_row >= 64 ? 32 : vec_per_row >= 32 ? 16 : 8;     // lanes per row: every lane gets at least two vectors
    const long long rows_per_block = (long long)kWarpsPerBlock * (32 / lpr);
    long long want = (total + rows_per_block - 1) / rows_per_block;
    const long long cap = (long long)sm_count() * kBlocksPerSM;
    int grid = (int)(want < cap ? want : cap);
    uint4 *c = reinterpret_cast<uint4 *>(cache);
    const uint4 *rw = reinterpret_cast<const uint4 *>(rows);
    const int full = (flags & ASTRAEA_SCATTER_SRC_FULL) ? 1 : 0;
    if (lpr == 32) scatter_kernel<32><<<grid, kWarpsPerBlock * 32, 0, stream>>>(c, rw, idx, B, N, M, vec_per_row, pitch_vec, full, err_word);
    else if (lpr == 16) scatter_kernel<16><<<grid, kWarpsPerBlock * 32, 0, stream>>>(c, rw, idx, B, N, M, vec_per_row, pitch_vec, full, err_word);
    else scatter_kernel<8><<<grid, kWarpsPerBlock * 32, 0, stream>>>(c, rw, idx, B, N, M, vec_per_row, pitch_vec, full, err_word);
    return check_launch("astraea_scatter_reuse");
}

}  // namespace astraea
