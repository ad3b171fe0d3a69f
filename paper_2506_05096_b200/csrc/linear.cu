// astraea_gathered_linear: y[b, i, :] = x[b, i, :] W^T + bias for the listed token rows i = idx[b, r];
// the other rows of y keep the cached result (Algorithm 1 lines 4-7 applied to a linear layer of the
// block: the query projection of the selected tokens, the output projection and the MLP on selected
// rows; with idx == NULL the key / value projections of all tokens).
//
// A dense contraction, so it runs on the tcgen05 tensor cores.  Persistent CTAs, one per SM, walk over
// 256-row x 256-column output tiles (column tiles of one row tile are neighbours in the walk, so the
// gathered rows stay in L2 while W, which is small, lives there anyway).  A tile is two 128-row sub-tiles
// that share every W tile in shared memory.  Warp roles:
//   warps 0-15  epilogue: two threads per output row (128 columns each); TMEM -> registers -> (+ bias, GELU, gate,
//               residual) -> bf16 -> the row of y that idx names (fused scatter);
//   warps 16-23 gather of the A operand: the listed rows of x, 64 columns (128 bytes) per pipeline stage,
//               by 16-byte cp.async into the 128-byte-swizzled layout the MMA reads (rows past the end
//               are zero-filled); the copies arrive on the stage's barrier by themselves, so a thread never
//               waits for its own copies, only for a free stage;
//   warp 24     TMA producer of the B operand: a 256 x 64 tile of W per stage (rows past N_out read as zero);
//   warp 25     tcgen05.mma issuer: per stage four 128 x 256 x 16 SS MMAs into each sub-tile's accumulator.
// Stages: 3 x (2 x 16 KB of A + 32 KB of W); TMEM: two accumulators of 256 columns.  Every mbarrier wait
// is bounded; on a timeout the CTA raises the error word, the remaining waits return at once, and the
// CTA runs out.
#include "common.cuh"
#include "sm100_ptx.cuh"
#include "bounded_wait.cuh"

namespace astraea {
namespace {

using namespace ptx;

// 128-row sub-tiles of a CTA tile, each with its own 256-column accumulator.  Two: a 256 x 256 tile reads 128 flop
// per byte of operands from L2 instead of 85, which is what bounds this kernel; it fills TMEM, so the epilogue is
// not hidden under the next main loop any more, and is still 4-15 % faster than one sub-tile with two accumulator sets.
constexpr int kMSub = 2;
constexpr int kBM = 128 * kMSub, kBN = 256, kBK = 64;
constexpr int kStages = (kMSub == 2) ? 3 : 4;
constexpr int kAccSets = 2 / kMSub;                      // accumulator sets in TMEM: two sets let the epilogue run under the next main loop
constexpr int kASubBytes = 128 * kBK * 2, kABytes = kMSub * kASubBytes, kBBytes = kBN * kBK * 2;
// Epilogue warps: four per sub-tile cover its 128 rows (one TMEM lane quarter each); kEpiSplit such groups share the 256
// columns of the accumulator.  Two: the epilogue is not hidden under the next tile's main loop (TMEM is full), so its
// time counts in full, and bias, GELU (erf), gate and residual make it a third to a half of a tile's time with one group.
constexpr int kEpiSplit = 2;
constexpr int kEpiWarps = 4 * kMSub * kEpiSplit, kGatherWarps = 4 * kMSub;
constexpr int kThreads = (kEpiWarps + kGatherWarps + 2) * 32;
constexpr int kTmaWarp = kEpiWarps + kGatherWarps, kMmaWarp = kTmaWarp + 1;
constexpr int kEpiStageBytes = 32 * 64;                  // per epilogue warp: 32 rows x 32 bf16 columns on their way to / from global memory
constexpr int kSmemBytes = kStages * (kABytes + kBBytes) + 256 + kEpiWarps * kEpiStageBytes + 1024;
static_assert(kSmemBytes <= 227 * 1024, "shared memory of one CTA");
constexpr uint32_t kAccCols = kBN, kTmemCols = 2 * kBN;

struct LinParams {
    const __nv_bfloat16 *x;
    const int32_t *idx;
    int M;                       // rows listed per batch element (N when idx == nullptr)
    const __nv_bfloat16 *bias;
    __nv_bfloat16 *y;
    int B, N, K, N_out;
    int compact;                 // y is [B, M, N_out]
    int compact_in;              // x is [B, M, K]
    int gelu;                    // y = GELU(x W^T + bias), exact (erf) form
    const __nv_bfloat16 *residual;   // added to the result after the gate; [B, N, N_out] rows at idx, or compact [B, M, N_out]
    int res_compact;
    const __nv_bfloat16 *gate;       // [B, N_out]: multiplies act(x W^T + bias) before the residual is added
    int *err_word;
};

__device__ __forceinline__ void cp_async_16(uint32_t dst, const void *src, bool valid) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(valid ? 16 : 0) : "memory");
}
// arrive on the mbarrier once every cp.async this thread has issued so far has landed (the arrival is one of
// those the barrier was initialised to expect)
__device__ __forceinline__ void cp_async_arrive(uint32_t bar) {
    asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(bar) : "memory");
}

// erf(x) to 1.5e-7 absolute (rational approximation 7.1.26 of Abramowitz and Stegun: 1 - (a1 t + ... + a5 t^5) e^{-x^2},
// t = 1 / (1 + p |x|)): two XU operations and nine FMA-pipe ones without a branch, about half of erff()'s cost, which
// counts because the epilogue of a tile is not hidden.  The result goes into a bf16 (2^-9 relative).
__device__ __forceinline__ float erf_fast(float x) {
    const float ax = fabsf(x);
    float t, e;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(t) : "f"(fmaf(0.3275911f, ax, 1.0f)));
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(ax * ax * -1.4426950408889634f));
    float pl = fmaf(1.061405429f, t, -1.453152027f);
    pl = fmaf(pl, t, 1.421413741f);
    pl = fmaf(pl, t, -0.284496736f);
    pl = fmaf(pl, t, 0.254829592f);
    return copysignf(fmaf(-pl * t, e, 1.0f), x);
}

// 2-D tiled load global -> shared, completion counted in bytes on an mbarrier
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *m, uint32_t bar, int c0, int c1) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(m), "r"(bar), "r"(c0), "r"(c1) : "memory");
}

// row of x that holds the g-th listed row (all batch elements in one list): -1 past the end, -2 for an index
// outside [0, N) or one that does not exceed its predecessor; *out_row is the row of y it goes to, *res_row the row
// of the residual, *batch the batch element
__device__ __forceinline__ long long source_row(const LinParams &p, long long g, long long total, long long *out_row,
                                                long long *res_row = nullptr, int *batch = nullptr) {
    if (g >= total) return -1;
    const int b = (int)(g / p.M), r = (int)(g - (long long)b * p.M);
    const int tok = p.idx ? __ldg(p.idx + g) : r;
    if ((unsigned)tok >= (unsigned)p.N) return -2;
    if (p.idx && r > 0 && __ldg(p.idx + g - 1) >= tok) return -2;      // not strictly ascending: a row would be written twice
    if (out_row) *out_row = p.compact ? g : (long long)b * p.N + tok;
    if (res_row) *res_row = p.res_compact ? g : (long long)b * p.N + tok;
    if (batch) *batch = b;
    return p.compact_in ? g : (long long)b * p.N + tok;
}

__global__ void __launch_bounds__(kThreads, 1)
gathered_linear_kernel(const __grid_constant__ CUtensorMap tmap_w, const LinParams p)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;

    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sA = smem_base, sB = sA + kStages * kABytes, bars = sB + kStages * kBBytes;
    const uint32_t bar_full = bars, bar_empty = bars + 8 * kStages, bar_acc_full = bars + 16 * kStages,
                   bar_acc_empty = bar_acc_full + 16;

    const int tid = threadIdx.x;
    const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);        // warp-uniform
    const int lane = tid & 31;
    const long long total_rows = (long long)p.B * p.M;
    const int tiles_m = (int)((total_rows + kBM - 1) / kBM), tiles_n = (p.N_out + kBN - 1) / kBN;
    const int total_tiles = tiles_m * tiles_n, k_steps = p.K / kBK;

    if (tid == 0) {
        abort_flag = 0;
        for (int s = 0; s < kStages; ++s) {
            mbar_init(bar_full + 8 * s, kGatherWarps * 32 + 1);     // every gather thread + the TMA producer
            mbar_init(bar_empty + 8 * s, 1);
        }
        for (int a = 0; a < kAccSets; ++a) { mbar_init(bar_acc_full + 8 * a, 1); mbar_init(bar_acc_empty + 8 * a, kEpiWarps * 32); }
        fence_barrier_init();
    }
    if (warp == kMmaWarp) {
        tmem_alloc(smem_u32(&tmem_slot), kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_slot;

    if (warp < kEpiWarps) {
        // ------------------------------------------------ epilogue
        // row of the CTA tile: sub-tile (warp / 4) % kMSub, TMEM lanes by warp % 4; columns [c0, c0 + kBN / kEpiSplit) by warp / (4 kMSub)
        const int sub = (warp >> 2) % kMSub, part = warp / (4 * kMSub);
        const int row = sub * 128 + (warp & 3) * 32 + lane;
        const int c0 = part * (kBN / kEpiSplit);
        const uint32_t t_row = tmem + ((uint32_t)((warp & 3) * 32) << 16) + sub * kAccCols;
        uint8_t *stage = smem_raw + (bars + 256 - smem_u32(smem_raw)) + warp * kEpiStageBytes;
        int it = 0;
        for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x, ++it) {
            const int tm = tile / tiles_n, tn = tile - tm * tiles_n;
            const int acc = it % kAccSets, n0 = tn * kBN;
            long long out_row = -1, res_row = -1;
            int batch = 0;
            const long long src = source_row(p, (long long)tm * kBM + row, total_rows, &out_row, &res_row, &batch);
            if (src == -2 && tn == 0 && part == 0) atomicExch(p.err_word, kErrBadIndex);
            if (src < 0) { out_row = -1; res_row = -1; }
            if (!p.residual) res_row = -1;
            const __nv_bfloat16 *gate = p.gate ? p.gate + (long long)batch * p.N_out : nullptr;
            wait_bar(bar_acc_full + 8 * acc, (it / kAccSets) & 1, &abort_flag, p.err_word);
            tc_fence_after();
            if (abort_flag) out_row = -1;
            // Global memory is touched in a transposed layout: a thread owns a row of the accumulator, so a warp that
            // stored its rows directly would touch 32 lines per instruction, 16 bytes in each (measured: ~9 us of a
            // 36 us tile, 16 us with a residual).  Instead lane l moves the 16-byte piece l & 3 of rows (l >> 2) + 8 j:
            // 64 contiguous bytes per row, 8 rows per instruction, through 2 KB of shared memory per warp (pieces
            // swizzled by the row so that both directions are free of bank conflicts).
            const int q = lane & 3;
#pragma unroll 1
            for (int c = c0; c < c0 + kBN / kEpiSplit; c += 32) {
                const int colq = n0 + c + q * 8;                    // the 8 columns this lane moves
                uint32_t rw[16];                                    // this thread's row of the residual: 32 bf16
                if (p.residual) {
                    uint4 rr[4];
#pragma unroll
                    for (int jj = 0; jj < 4; ++jj) {
                        const int r = (lane >> 2) + 8 * jj;
                        const long long rrow = __shfl_sync(0xffffffffu, res_row, r);
                        rr[jj] = (rrow >= 0 && colq < p.N_out) ? __ldg(reinterpret_cast<const uint4 *>(p.residual + rrow * p.N_out + colq))
                                                                : make_uint4(0, 0, 0, 0);
                    }
#pragma unroll
                    for (int jj = 0; jj < 4; ++jj) {
                        const int r = (lane >> 2) + 8 * jj;
                        *reinterpret_cast<uint4 *>(stage + r * 64 + ((q ^ ((r >> 1) & 3)) << 4)) = rr[jj];
                    }
                    __syncwarp();
#pragma unroll
                    for (int v = 0; v < 4; ++v) {
                        const uint4 t = *reinterpret_cast<const uint4 *>(stage + lane * 64 + ((v ^ ((lane >> 1) & 3)) << 4));
                        rw[4 * v] = t.x; rw[4 * v + 1] = t.y; rw[4 * v + 2] = t.z; rw[4 * v + 3] = t.w;
                    }
                    __syncwarp();
                }
                uint32_t o[32];
                tmem_ld32(t_row + acc * kMSub * kAccCols + c, o);
                tc_wait_ld();
                if (c + 32 == c0 + kBN / kEpiSplit) {    // this thread's part of the accumulator has been read: the MMA warp may reuse it
                    tc_fence_before();
                    mbar_arrive(bar_acc_empty + 8 * acc);
                }
#pragma unroll
                for (int v = 0; v < 4; ++v) {
                    const int col = n0 + c + v * 8;
                    float f[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) f[i] = __uint_as_float(o[v * 8 + i]);
                    if (col < p.N_out) {                 // N_out is a multiple of 8; columns past it are never stored
                        if (p.bias) {
                            const uint4 bb = __ldg(reinterpret_cast<const uint4 *>(p.bias + col));
                            const uint32_t bw[4] = {bb.x, bb.y, bb.z, bb.w};
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                f[2 * i] += __uint_as_float(bw[i] << 16);
                                f[2 * i + 1] += __uint_as_float(bw[i] & 0xffff0000u);
                            }
                        }
                        if (p.gelu) {
#pragma unroll
                            for (int i = 0; i < 8; ++i) f[i] = 0.5f * f[i] * (1.0f + erf_fast(f[i] * 0.70710678118654752f));
                        }
                        if (gate) {
                            const uint4 gg = __ldg(reinterpret_cast<const uint4 *>(gate + col));
                            const uint32_t gw[4] = {gg.x, gg.y, gg.z, gg.w};
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                f[2 * i] *= __uint_as_float(gw[i] << 16);
                                f[2 * i + 1] *= __uint_as_float(gw[i] & 0xffff0000u);
                            }
                        }
                        if (p.residual) {
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                f[2 * i] += __uint_as_float(rw[4 * v + i] << 16);
                                f[2 * i + 1] += __uint_as_float(rw[4 * v + i] & 0xffff0000u);
                            }
                        }
                    }
                    uint32_t w[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        __nv_bfloat162 v2 = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
                        w[i] = *reinterpret_cast<uint32_t *>(&v2);
                    }
                    *reinterpret_cast<uint4 *>(stage + lane * 64 + ((v ^ ((lane >> 1) & 3)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
                }
                __syncwarp();
#pragma unroll
                for (int jj = 0; jj < 4; ++jj) {
                    const int r = (lane >> 2) + 8 * jj;
                    const long long orow = __shfl_sync(0xffffffffu, out_row, r);
                    const uint4 t = *reinterpret_cast<const uint4 *>(stage + r * 64 + ((q ^ ((r >> 1) & 3)) << 4));
                    if (orow >= 0 && colq < p.N_out) *reinterpret_cast<uint4 *>(p.y + orow * p.N_out + colq) = t;
                }
                __syncwarp();
            }
        }
    } else if (warp < kEpiWarps + kGatherWarps) {
        // ------------------------------------------------ gather of the A rows (cp.async, 128-byte swizzle)
        const int t = tid - kEpiWarps * 32;                   // 0 .. 128 kMSub - 1
        const int chunk = t & 7, row0 = t >> 3;               // this thread: 16-byte chunk `chunk` of rows row0 + 16 kMSub i
        int g = 0;                                            // running stage count over all tiles
        for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x) {
            const int tm = tile / tiles_n;
            const __nv_bfloat16 *src[8];
            uint32_t off[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int r = row0 + 16 * kMSub * i;
                const long long s = source_row(p, (long long)tm * kBM + r, total_rows, nullptr);
                src[i] = (s >= 0) ? p.x + s * p.K + chunk * 8 : nullptr;
                off[i] = (r >> 7) * kASubBytes + (r & 127) * 128 + ((chunk ^ (r & 7)) << 4);
            }
            for (int ks = 0; ks < k_steps; ++ks, ++g) {
                const int st = g % kStages;
                wait_bar(bar_empty + 8 * st, ((g / kStages) & 1) ^ 1, &abort_flag, p.err_word);
#pragma unroll
                for (int i = 0; i < 8; ++i)
                    cp_async_16(sA + st * kABytes + off[i], src[i] ? (const void *)(src[i] + ks * kBK) : (const void *)p.x, src[i] != nullptr);
                cp_async_arrive(bar_full + 8 * st);           // asynchronous: the thread goes on to the next free stage
            }
        }
    } else if (warp == kTmaWarp) {
        // ------------------------------------------------ TMA producer of the W tiles
        if (elect_one()) prefetch_tensormap(&tmap_w);
        int g = 0;
        for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x) {
            const int tn = tile % tiles_n;
            for (int ks = 0; ks < k_steps; ++ks, ++g) {
                const int st = g % kStages;
                wait_bar(bar_empty + 8 * st, ((g / kStages) & 1) ^ 1, &abort_flag, p.err_word);
                if (elect_one()) {
                    mbar_arrive_expect_tx(bar_full + 8 * st, kBBytes);
                    tma_load_2d(sB + st * kBBytes, &tmap_w, bar_full + 8 * st, ks * kBK, tn * kBN);
                }
                __syncwarp();
            }
        }
        // every copy issued above must have landed before the CTA's shared memory is released
        for (int gs = (g > kStages ? g - kStages : 0); gs < g; ++gs)
            wait_bar(bar_full + 8 * (gs % kStages), (gs / kStages) & 1, &abort_flag, p.err_word);
    } else {
        // ------------------------------------------------ MMA issuer
        constexpr uint32_t idesc = idesc_bf16(128, kBN, false);
        int g = 0, it = 0;
        for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x, ++it) {
            const int acc = it % kAccSets;
            wait_bar(bar_acc_empty + 8 * acc, ((it / kAccSets) & 1) ^ 1, &abort_flag, p.err_word);
            for (int ks = 0; ks < k_steps; ++ks, ++g) {
                const int st = g % kStages;
                wait_bar(bar_full + 8 * st, (g / kStages) & 1, &abort_flag, p.err_word);
                fence_proxy_async_smem();             // the gathered rows were written through the generic proxy
                tc_fence_after();
                if (elect_one()) {
#pragma unroll
                    for (int kk = 0; kk < kBK / 16; ++kk) {
#pragma unroll
                        for (int sub = 0; sub < kMSub; ++sub)       // the sub-tiles share the W tile in shared memory
                            mma_ss(tmem + (acc * kMSub + sub) * kAccCols,
                                   smem_desc(sA + st * kABytes + sub * kASubBytes + kk * 32, 16, 1024, kSwizzle128B),
                                   smem_desc(sB + st * kBBytes + kk * 32, 16, 1024, kSwizzle128B),
                                   idesc, (ks > 0 || kk > 0) ? 1u : 0u);
                    }
                    tc_commit(bar_empty + 8 * st);
                    if (ks == k_steps - 1) tc_commit(bar_acc_full + 8 * acc);
                }
                __syncwarp();
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == kMmaWarp) tmem_dealloc(tmem, kTmemCols);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

}  // namespace

size_t linear_workspace_bytes() { return 256; }

int32_t launch_gathered_linear(const void *x, const int32_t *idx, int M, const void *w, const void *bias, void *y,
                               int B, int N, int K, int N_out, uint32_t flags, int *err_word, cudaStream_t stream,
                               const void *residual, const void *gate)
{
    const EncodeTiledFn enc = reinterpret_cast<EncodeTiledFn>(tensor_map_encoder());
    if (!enc) return fail(ASTRAEA_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
    // W as a 2-D tensor (K, N_out) with 128-byte-swizzled boxes of 64 columns x 256 rows
    CUtensorMap mw;
    cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)N_out};
    cuuint64_t strides[1] = {(cuuint64_t)K * 2};
    cuuint32_t box[2] = {(cuuint32_t)kBK, (cuuint32_t)kBN};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = enc(&mw, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(w), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(ASTRAEA_ERR_INVALID_ARG, "astraea_gathered_linear: tensor map of W rejected (CUresult %d)", (int)r);
    static PerDeviceOnce attrs;                   // the attribute is per device
    if (attrs.run([] { return cudaFuncSetAttribute(gathered_linear_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes); }) != cudaSuccess)
        return check_launch("astraea_gathered_linear (shared memory attribute)");
    LinParams p;
    p.x = reinterpret_cast<const __nv_bfloat16 *>(x);
    p.idx = idx;
    p.M = idx ? M : N;
    p.bias = reinterpret_cast<const __nv_bfloat16 *>(bias);
    p.y = reinterpret_cast<__nv_bfloat16 *>(y);
    p.B = B; p.N = N; p.K = K; p.N_out = N_out;
    p.compact = (flags & ASTRAEA_LINEAR_COMPACT_OUT) ? 1 : 0;
    p.compact_in = (flags & ASTRAEA_LINEAR_COMPACT_IN) ? 1 : 0;
    p.gelu = (flags & ASTRAEA_LINEAR_GELU) ? 1 : 0;
    p.residual = reinterpret_cast<const __nv_bfloat16 *>(residual);
    p.res_compact = (flags & ASTRAEA_LINEAR_COMPACT_RES) ? 1 : 0;
    p.gate = reinterpret_cast<const __nv_bfloat16 *>(gate);
    p.err_word = err_word;
    const long long rows = (long long)B * p.M;
    const long long tiles = ((rows + kBM - 1) / kBM) * ((N_out + kBN - 1) / kBN);
    const int n_sm = sm_count();
    const int grid = (int)(tiles < n_sm ? tiles : n_sm);
    gathered_linear_kernel<<<grid, kThreads, kSmemBytes, stream>>>(mw, p);
    return check_launch("astraea_gathered_linear");
}

}  // namespace astraea
