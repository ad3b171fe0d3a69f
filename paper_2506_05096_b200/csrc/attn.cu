// astraea_sparse_attn: out[i] = Softmax(q_i K^T * scale) V for the selected query rows i
// against ALL keys/values, written in place over the cached output (Algorithm 1 lines 6-7;
// Section 3.2 "Sparse Attention").
//
// One CTA per (256 selected queries, head, batch): two 128-row query tiles that share every
// K/V tile of 64 keys.  Warp roles (320 threads):
//   warps 0-3 / 4-7  softmax of query tile 0 / 1: gather the tile's Q rows into 128B-swizzled
//              shared memory, then per key tile read S from TMEM (one thread per query row),
//              online softmax in the log2 domain with lazy rescaling of O, write P (bf16) back
//              to TMEM over S, and at the end normalise O and scatter it to the rows q_idx names;
//   warp 8     TMA producer: K and V tiles into multi-stage swizzled buffers;
//   warp 9     tcgen05.mma issuer: S = Q K^T (SS, K-major operands), O += P V (P from TMEM,
//              V as an MN-major shared-memory operand); owns the TMEM allocation.
// S is double-buffered per query tile, so the QK^T of key tile j+1 is already in TMEM while the
// softmax of tile j runs: the softmax warps never wait for the tensor core in steady state.
// TMEM columns: S/P of (tile t, buffer u) at (2t+u)*64; O of tile t at 256 + 128 t.
// The producer and issuer warps run warp-uniform code and elect one lane per instruction, so
// that descriptors and addresses stay in uniform registers (a lone diverged thread issues
// tcgen05.mma several times slower).  Every mbarrier wait is bounded; on a timeout the CTA
// raises the error word, the remaining waits return at once, and the CTA runs out.
#include "common.cuh"
#include "sm100_ptx.cuh"

namespace astraea {
namespace {

using namespace ptx;

constexpr int kBlockM = 128;                     // rows of one query tile
constexpr int kTilesM = 2;                       // query tiles per CTA
constexpr int kBlockN = 64;                      // keys per K/V tile
constexpr int kThreads = 320;
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kColO = 256;
constexpr float kRescaleThreshold = 8.0f;        // log2 units: P stays below 2^8
constexpr uint64_t kWaitLimitNs = 1000000000ull; // bounded waits: one second

template <int DH> struct Cfg {
    static constexpr int kChunks = DH / 64;                       // 64-column (128-byte) swizzle chunks
    static constexpr int kQChunkBytes = kBlockM * 128;            // 128 query rows x 128 bytes
    static constexpr int kQTileBytes = kChunks * kQChunkBytes;
    static constexpr int kChunkBytes = kBlockN * 128;             // 64 keys x 128 bytes
    static constexpr int kTileBytes = kChunks * kChunkBytes;      // one K or V tile
    static constexpr int kStagesK = (DH == 128) ? 5 : 6;
    static constexpr int kStagesV = (DH == 128) ? 5 : 6;
    static constexpr int kBarBytes = 512;
    static constexpr int kSmemBytes = kQTileBytes * kTilesM + kTileBytes * (kStagesK + kStagesV) + kBarBytes + 1024;
};

struct Params {
    const __nv_bfloat16 *q;
    int64_t q_sb, q_sh, q_sn;
    const int32_t *q_idx;
    int M;
    __nv_bfloat16 *out;
    float *lse_out;
    int N, H;
    float scale, scale_log2;
    int compact;
    int *err_word;
};

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ bool elect_one() {
    uint32_t pred;
    asm volatile("{\n\t.reg .pred px;\n\telect.sync _|px, 0xffffffff;\n\tselp.u32 %0, 1, 0, px;\n\t}" : "=r"(pred));
    return pred != 0;
}

// Bounded mbarrier wait.  Gives up after the limit, or at once when another wait of this CTA
// already gave up; the caller carries on (its results are void, the error word says so).
__device__ __forceinline__ void wait_bar(uint32_t bar, uint32_t parity, volatile int *abort_flag, int *err_word) {
    if (mbar_try_wait(bar, parity)) return;
    if (*abort_flag) return;
    const uint64_t t0 = globaltimer_ns();
    uint32_t spins = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++spins & 255u) == 0) {
            if (*abort_flag) return;
            if (globaltimer_ns() - t0 > kWaitLimitNs) {
                *abort_flag = 1;
                atomicExch(err_word, kErrTimeout);
                return;
            }
        }
    }
}

struct Bars {
    uint32_t q, o;                  // [kTilesM]
    uint32_t s, p;                  // [kTilesM][2]
    uint32_t kf, ke, vf, ve;        // [stages]
};

// ---------------------------------------------------------------- softmax warpgroup (one query tile)
template <int DH>
__device__ __forceinline__ void softmax_role(const Params &p, const Bars &bar, int tile, uint8_t *sQ_gen, uint32_t tmem,
                                             int m_base, int h, int b, int n_tiles, volatile int *abort_flag)
{
    using C = Cfg<DH>;
    const int wtid = threadIdx.x & 127, lane = wtid & 31;
    const int warp = __shfl_sync(0xffffffffu, wtid >> 5, 0);       // warp-uniform
    // gather this tile's Q rows (swizzled, K-major)
    constexpr int kVecPerRow = DH / 8;                 // 16-byte vectors per row
    constexpr int kRowsPerIter = 32 / kVecPerRow;
    {
        const int sub = lane / kVecPerRow, c = lane % kVecPerRow;
#pragma unroll 4
        for (int r0 = warp * kRowsPerIter; r0 < kBlockM; r0 += 4 * kRowsPerIter) {
            const int r = r0 + sub;
            const int m = m_base + r;
            uint4 val = make_uint4(0, 0, 0, 0);
            if (m < p.M) {
                const int tok = p.q_idx ? __ldg(p.q_idx + (size_t)b * p.M + m) : m;
                if ((unsigned)tok < (unsigned)p.N) {
                    const __nv_bfloat16 *src = p.q + (size_t)b * p.q_sb + (size_t)tok * p.q_sn + (size_t)h * p.q_sh + c * 8;
                    val = __ldg(reinterpret_cast<const uint4 *>(src));
                }
            }
            const uint32_t off = (c >> 3) * C::kQChunkBytes + r * 128 + (((c & 7) ^ (r & 7)) << 4);
            *reinterpret_cast<uint4 *>(sQ_gen + off) = val;
        }
    }
    fence_proxy_async_smem();
    mbar_arrive(bar.q + 8 * tile);

    const uint32_t t_row = tmem + ((uint32_t)(warp * 32) << 16);
    const uint32_t t_s0 = t_row + tile * 128;
    const uint32_t t_o = t_row + kColO + tile * 128;
    const uint32_t bar_s = bar.s + 16 * tile, bar_p = bar.p + 16 * tile, bar_o = bar.o + 8 * tile;
    const int m = m_base + wtid;
    int tok = -1;
    if (m < p.M) {
        tok = p.q_idx ? __ldg(p.q_idx + (size_t)b * p.M + m) : m;
        if ((unsigned)tok >= (unsigned)p.N) { atomicExch(p.err_word, kErrBadIndex); tok = -1; }
    }
    const float sl2 = p.scale_log2;
    float m_ref = -INFINITY, l_sum = 0.f;

    for (int j = 0; j < n_tiles; ++j) {
        const int buf = j & 1;
        const uint32_t t_s = t_s0 + buf * kBlockN;
        wait_bar(bar_s + 8 * buf, (j >> 1) & 1, abort_flag, p.err_word);
        tc_fence_after();
        float s[kBlockN];
        {
            uint32_t t0[32], t1[32];
            tmem_ld32(t_s, t0);
            tmem_ld32(t_s + 32, t1);
            tc_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                s[i] = __uint_as_float(t0[i]);
                s[32 + i] = __uint_as_float(t1[i]);
            }
        }
        const int valid = p.N - j * kBlockN;           // keys of this tile that exist
        if (valid < kBlockN) {
#pragma unroll
            for (int i = 0; i < kBlockN; ++i) if (i >= valid) s[i] = -INFINITY;
        }
        // row maximum: independent partial maxima keep the dependency chains short
        float mx4[4] = {s[0], s[1], s[2], s[3]};
#pragma unroll
        for (int i = 4; i < kBlockN; i += 4) {
            mx4[0] = fmaxf(mx4[0], s[i]); mx4[1] = fmaxf(mx4[1], s[i + 1]);
            mx4[2] = fmaxf(mx4[2], s[i + 2]); mx4[3] = fmaxf(mx4[3], s[i + 3]);
        }
        const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));

        if (j == 0) {
            m_ref = mx;
        } else {
            const bool need = (mx - m_ref) * sl2 > kRescaleThreshold;
            if (__any_sync(0xffffffffu, need)) {
                float alpha = 1.0f;
                if (need) { alpha = ex2((m_ref - mx) * sl2); m_ref = mx; l_sum *= alpha; }
                wait_bar(bar_o, (j - 1) & 1, abort_flag, p.err_word);     // P V of the previous key tile has landed
                tc_fence_after();
#pragma unroll
                for (int cc = 0; cc < DH / 32; ++cc) {
                    uint32_t o[32];
                    tmem_ld32(t_o + cc * 32, o);
                    tc_wait_ld();
#pragma unroll
                    for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
                    tmem_st32(t_o + cc * 32, o);
                }
                tc_wait_st();
            }
        }
        const float neg = -m_ref * sl2;
        float sum4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int i = 0; i < kBlockN; i += 4) {
#pragma unroll
            for (int u = 0; u < 4; ++u) { s[i + u] = ex2(fmaf(s[i + u], sl2, neg)); sum4[u] += s[i + u]; }
        }
        l_sum += (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);
        // P as bf16 pairs over the first 32 columns of this S buffer (element 2c in the low half)
        {
            uint32_t pk[32];
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                __nv_bfloat162 v2 = __floats2bfloat162_rn(s[2 * i], s[2 * i + 1]);
                pk[i] = *reinterpret_cast<uint32_t *>(&v2);
            }
            tmem_st32(t_s, pk);
        }
        tc_wait_st();
        tc_fence_before();
        mbar_arrive(bar_p + 8 * buf);
    }

    // epilogue: normalise and scatter
    wait_bar(bar_o, (n_tiles - 1) & 1, abort_flag, p.err_word);
    tc_fence_after();
    const float inv_l = 1.0f / l_sum;
    __nv_bfloat16 *dst = nullptr;
    if (tok >= 0 && !*abort_flag) {
        const size_t orow = p.compact ? ((size_t)b * p.M + m) : ((size_t)b * p.N + tok);
        dst = p.out + (orow * p.H + h) * DH;
        if (p.lse_out) {
            const size_t li = p.compact ? (((size_t)b * p.H + h) * p.M + m) : (((size_t)b * p.H + h) * p.N + tok);
            p.lse_out[li] = m_ref * p.scale + logf(l_sum);
        }
    }
#pragma unroll
    for (int cc = 0; cc < DH / 32; ++cc) {
        uint32_t o[32];
        tmem_ld32(t_o + cc * 32, o);
        tc_wait_ld();
        if (dst) {
#pragma unroll
            for (int v = 0; v < 4; ++v) {
                uint32_t w[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    __nv_bfloat162 v2 = __floats2bfloat162_rn(__uint_as_float(o[v * 8 + 2 * i]) * inv_l,
                                                              __uint_as_float(o[v * 8 + 2 * i + 1]) * inv_l);
                    w[i] = *reinterpret_cast<uint32_t *>(&v2);
                }
                *reinterpret_cast<uint4 *>(dst + cc * 32 + v * 8) = make_uint4(w[0], w[1], w[2], w[3]);
            }
        }
    }
}

template <int DH>
__global__ void __launch_bounds__(kThreads, 1)
sparse_attn_kernel(const __grid_constant__ CUtensorMap tmap_k, const __grid_constant__ CUtensorMap tmap_v, const Params p)
{
    using C = Cfg<DH>;
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;

    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    const uint32_t sQ = smem_base;
    const uint32_t sK = sQ + kTilesM * C::kQTileBytes;
    const uint32_t sV = sK + C::kStagesK * C::kTileBytes;
    const uint32_t bars = sV + C::kStagesV * C::kTileBytes;
    Bars bar;
    bar.q = bars; bar.o = bars + 16; bar.s = bars + 32; bar.p = bars + 64;
    bar.kf = bars + 96;
    bar.ke = bar.kf + 8 * C::kStagesK;
    bar.vf = bar.ke + 8 * C::kStagesK;
    bar.ve = bar.vf + 8 * C::kStagesV;
    static_assert(96 + 16 * (C::kStagesK + C::kStagesV) <= C::kBarBytes, "barrier area too small");

    const int tid = threadIdx.x;
    const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);        // warp-uniform
    const int m0 = blockIdx.x * (kTilesM * kBlockM), h = blockIdx.y, b = blockIdx.z;
    const int n_tiles = (p.N + kBlockN - 1) / kBlockN;

    if (tid == 0) {
        abort_flag = 0;
        for (int t = 0; t < kTilesM; ++t) {
            mbar_init(bar.q + 8 * t, 128); mbar_init(bar.o + 8 * t, 1);
            for (int u = 0; u < 2; ++u) { mbar_init(bar.s + 16 * t + 8 * u, 1); mbar_init(bar.p + 16 * t + 8 * u, 128); }
        }
        for (int s = 0; s < C::kStagesK; ++s) { mbar_init(bar.kf + 8 * s, 1); mbar_init(bar.ke + 8 * s, 1); }
        for (int s = 0; s < C::kStagesV; ++s) { mbar_init(bar.vf + 8 * s, 1); mbar_init(bar.ve + 8 * s, 1); }
        fence_barrier_init();
    }
    if (warp == 9) {
        tmem_alloc(smem_u32(&tmem_slot), kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_slot;

    if (warp < 8) {
        const int tile = warp >> 2;
        softmax_role<DH>(p, bar, tile, smem_gen + tile * C::kQTileBytes, tmem, m0 + tile * kBlockM, h, b, n_tiles, &abort_flag);
    } else if (warp == 8) {
        // ------------------------------------------------ TMA producer (warp-uniform, one elected lane issues)
        if (elect_one()) { prefetch_tensormap(&tmap_k); prefetch_tensormap(&tmap_v); }
        auto load_k = [&](int j) {
            const int st = j % C::kStagesK;
            wait_bar(bar.ke + 8 * st, ((j / C::kStagesK) & 1) ^ 1, &abort_flag, p.err_word);
            if (elect_one()) {
                mbar_arrive_expect_tx(bar.kf + 8 * st, C::kTileBytes);
#pragma unroll
                for (int ch = 0; ch < C::kChunks; ++ch)
                    tma_load_4d(sK + st * C::kTileBytes + ch * C::kChunkBytes, &tmap_k, bar.kf + 8 * st, ch * 64, j * kBlockN, h, b);
            }
            __syncwarp();
        };
        auto load_v = [&](int j) {
            const int st = j % C::kStagesV;
            wait_bar(bar.ve + 8 * st, ((j / C::kStagesV) & 1) ^ 1, &abort_flag, p.err_word);
            if (elect_one()) {
                mbar_arrive_expect_tx(bar.vf + 8 * st, C::kTileBytes);
#pragma unroll
                for (int ch = 0; ch < C::kChunks; ++ch)
                    tma_load_4d(sV + st * C::kTileBytes + ch * C::kChunkBytes, &tmap_v, bar.vf + 8 * st, ch * 64, j * kBlockN, h, b);
            }
            __syncwarp();
        };
        // K runs one tile ahead of V: K_{j+1} is needed before V_j
        load_k(0);
        for (int j = 0; j < n_tiles; ++j) {
            if (j + 1 < n_tiles) load_k(j + 1);
            load_v(j);
        }
        // every copy issued above must have landed before the CTA's shared memory is released
        for (int j = (n_tiles > C::kStagesK ? n_tiles - C::kStagesK : 0); j < n_tiles; ++j)
            wait_bar(bar.kf + 8 * (j % C::kStagesK), (j / C::kStagesK) & 1, &abort_flag, p.err_word);
        for (int j = (n_tiles > C::kStagesV ? n_tiles - C::kStagesV : 0); j < n_tiles; ++j)
            wait_bar(bar.vf + 8 * (j % C::kStagesV), (j / C::kStagesV) & 1, &abort_flag, p.err_word);
    } else {
        // ------------------------------------------------ MMA issuer (warp-uniform, one elected lane issues)
        constexpr uint32_t idesc_qk = idesc_bf16(kBlockM, kBlockN, false);
        constexpr uint32_t idesc_pv = idesc_bf16(kBlockM, DH, true);
        auto issue_qk = [&](int j) {                  // S[t][j&1] = Q_t K_j^T for both query tiles
            const int st = j % C::kStagesK;
            const uint32_t kbase = sK + st * C::kTileBytes;
            const uint32_t sbuf = (j & 1) * kBlockN;
            wait_bar(bar.kf + 8 * st, (j / C::kStagesK) & 1, &abort_flag, p.err_word);
            tc_fence_after();
            if (elect_one()) {
#pragma unroll
                for (int t = 0; t < kTilesM; ++t) {
#pragma unroll
                    for (int ks = 0; ks < DH / 16; ++ks)
                        mma_ss(tmem + t * 128 + sbuf,
                               smem_desc(sQ + t * C::kQTileBytes + (ks >> 2) * C::kQChunkBytes + (ks & 3) * 32, 16, 1024, kSwizzle128B),
                               smem_desc(kbase + (ks >> 2) * C::kChunkBytes + (ks & 3) * 32, 16, 1024, kSwizzle128B),
                               idesc_qk, ks > 0);
                    tc_commit(bar.s + 16 * t + 8 * (j & 1));
                }
                tc_commit(bar.ke + 8 * st);
            }
            __syncwarp();
        };
        wait_bar(bar.q, 0, &abort_flag, p.err_word);
        wait_bar(bar.q + 8, 0, &abort_flag, p.err_word);
        issue_qk(0);
        for (int j = 0; j < n_tiles; ++j) {
            if (j + 1 < n_tiles) issue_qk(j + 1);     // its S buffer held P of tile j-1, already consumed in order
            const int sv = j % C::kStagesV;
            const uint32_t vbase = sV + sv * C::kTileBytes;
            const uint32_t sbuf = (j & 1) * kBlockN;
            wait_bar(bar.vf + 8 * sv, (j / C::kStagesV) & 1, &abort_flag, p.err_word);
#pragma unroll
            for (int t = 0; t < kTilesM; ++t) {
                wait_bar(bar.p + 16 * t + 8 * (j & 1), (j >> 1) & 1, &abort_flag, p.err_word);
                tc_fence_after();
                if (elect_one()) {
#pragma unroll
                    for (int ks = 0; ks < kBlockN / 16; ++ks)
                        mma_ts(tmem + kColO + t * 128, tmem + t * 128 + sbuf + ks * 8,
                               smem_desc(vbase + ks * 2048, C::kChunkBytes, 1024, kSwizzle128B),
                               idesc_pv, (j > 0 || ks > 0) ? 1u : 0u);
                    tc_commit(bar.o + 8 * t);
                    if (t == kTilesM - 1) tc_commit(bar.ve + 8 * sv);
                }
                __syncwarp();
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 9) tmem_dealloc(tmem, kTmemCols);
}

// ------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
    }
    return fn;
}

// K or V as a 4-D tensor (d, N, H, B) with 128-byte-swizzled boxes of 64 columns x 128 tokens
int32_t make_kv_map(CUtensorMap *map, const void *base, int B, int H, int N, int d,
                    int64_t sb, int64_t sh, int64_t sn)
{
    EncodeTiledFn enc = get_encode_fn();
    if (!enc) return fail(ASTRAEA_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
    cuuint64_t dims[4] = {(cuuint64_t)d, (cuuint64_t)N, (cuuint64_t)H, (cuuint64_t)B};
    cuuint64_t strides[3] = {(cuuint64_t)sn * 2, (cuuint64_t)sh * 2, (cuuint64_t)sb * 2};
    cuuint32_t box[4] = {64, (cuuint32_t)kBlockN, 1, 1};   // 64 columns x one key tile
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(base), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(ASTRAEA_ERR_INVALID_ARG, "tensor map rejected (CUresult %d): check K/V strides and alignment", (int)r);
    return ASTRAEA_OK;
}

template <int DH>
int32_t launch_dh(const AttnArgs &a, cudaStream_t stream)
{
    using C = Cfg<DH>;
    CUtensorMap mk, mv;
    int32_t rc = make_kv_map(&mk, a.k, a.B, a.H, a.N, a.d, a.k_sb, a.k_sh, a.k_sn);
    if (rc != ASTRAEA_OK) return rc;
    rc = make_kv_map(&mv, a.v, a.B, a.H, a.N, a.d, a.v_sb, a.v_sh, a.v_sn);
    if (rc != ASTRAEA_OK) return rc;
    static bool attr_set = false;
    if (!attr_set) {
        if (cudaFuncSetAttribute(sparse_attn_kernel<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes) != cudaSuccess)
            return check_launch("astraea_sparse_attn (shared memory attribute)");
        attr_set = true;
    }
    Params p;
    p.q = reinterpret_cast<const __nv_bfloat16 *>(a.q);
    p.q_sb = a.q_sb; p.q_sh = a.q_sh; p.q_sn = a.q_sn;
    p.q_idx = a.q_idx; p.M = a.M;
    p.out = reinterpret_cast<__nv_bfloat16 *>(a.out);
    p.lse_out = a.lse_out;
    p.N = a.N; p.H = a.H;
    p.scale = a.scale;
    p.scale_log2 = a.scale * 1.4426950408889634f;
    p.compact = (a.flags & ASTRAEA_ATTN_COMPACT_OUT) ? 1 : 0;
    p.err_word = a.err_word;
    dim3 grid((a.M + kTilesM * kBlockM - 1) / (kTilesM * kBlockM), a.H, a.B);
    sparse_attn_kernel<DH><<<grid, kThreads, C::kSmemBytes, stream>>>(mk, mv, p);
    return check_launch("astraea_sparse_attn");
}

}  // namespace

size_t attn_workspace_bytes(int, int, int, int, int) { return 256; }

int32_t launch_sparse_attn(const AttnArgs &a, cudaStream_t stream)
{
    switch (a.d) {
    case 64: return launch_dh<64>(a, stream);
    case 128: return launch_dh<128>(a, stream);
    default: return fail(ASTRAEA_ERR_UNSUPPORTED, "head_dim %d is not supported", a.d);
    }
}

}  // namespace astraea
