// astraea_select: budgeted top-k per batch row (Algorithm 1 line 3), deterministic.
//
// Scores are mapped to order-preserving 32-bit keys (larger score -> larger key; -0 == +0;
// NaN ranks as -inf).  A most-significant-digit radix select (4 passes of 8 bits, histogram
// in shared memory) finds the key T of the k-th largest score and how many scores equal to
// T still belong to the selection.  One ordered pass then writes both index lists in
// ascending token order with a block-wide prefix scan (no atomics on output positions), so
// equal scores go to the lower index, and updates the skip counters.
//
// One CTA of 1024 threads per batch row; the score row (<= 0.5 MB) stays in L2 between
// passes.  The call is latency-bound, not bandwidth-bound, at the sizes of the workloads.
#include "common.cuh"

namespace astraea {
namespace {

constexpr int kThreads = 1024;
constexpr int kItems = 4;                       // consecutive tokens per thread in the ordered pass

__device__ __forceinline__ uint32_t score_key(float s) {
    uint32_t u = __float_as_uint(s);
    if ((u & 0x7fffffffu) > 0x7f800000u) u = 0xff800000u;      // NaN -> -inf
    if ((u << 1) == 0) u = 0;                                    // -0 -> +0
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

__global__ void __launch_bounds__(kThreads)
select_kernel(const float *__restrict__ score, int N_sel, int k, int n_always,
              int32_t *__restrict__ idx_sel, int32_t *__restrict__ idx_rem, int32_t *__restrict__ n_skip)
{
    __shared__ uint32_t hist[256];
    __shared__ uint32_t warp_tot[32];
    __shared__ uint32_t s_prefix, s_kk, s_chunk_tot;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b = blockIdx.x;
    const float *s = score + (size_t)b * N_sel;
    int32_t *sel = idx_sel ? idx_sel + (size_t)b * (k + n_always) : nullptr;
    int32_t *rem = idx_rem ? idx_rem + (size_t)b * (N_sel - k) : nullptr;
    int32_t *nsk = n_skip ? n_skip + (size_t)b * N_sel : nullptr;

    uint32_t T = 0xffffffffu;        // no key reaches this value
    uint32_t need_eq = 0;

    if (k > 0) {
        uint32_t prefix = 0, mask = 0, kk = (uint32_t)k;
        for (int shift = 24; shift >= 0; shift -= 8) {
            for (int i = tid; i < 256; i += kThreads) hist[i] = 0;
            __syncthreads();
            for (int i0 = 0; i0 < N_sel; i0 += kThreads) {
                int i = i0 + tid;
                bool live = false;
                uint32_t bin = 0;
                if (i < N_sel) {
                    uint32_t key = score_key(s[i]);
                    live = (key & mask) == prefix;
                    bin = (key >> shift) & 255u;
                }
                // one shared-memory atomic per distinct bin per warp
                uint32_t act = __ballot_sync(0xffffffffu, live);
                if (live) {
                    uint32_t peers = __match_any_sync(act, bin);
                    if (lane == (__ffs(peers) - 1)) atomicAdd(&hist[bin], (uint32_t)__popc(peers));
                }
            }
            __syncthreads();
            if (warp == 0) {
                // lane l owns bins 255-8l .. 248-8l (descending); find where the count from the top reaches kk
                uint32_t c[8], tot = 0;
#pragma unroll
                for (int j = 0; j < 8; ++j) { c[j] = hist[255 - 8 * lane - j]; tot += c[j]; }
                uint32_t inc = tot;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    uint32_t t = __shfl_up_sync(0xffffffffu, inc, o);
                    if (lane >= o) inc += t;
                }
                uint32_t exc = inc - tot;
                bool mine = (exc < kk) && (inc >= kk);
                if (mine) {
                    uint32_t above = exc;
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        if (above + c[j] >= kk) {
                            s_prefix = prefix | ((uint32_t)(255 - 8 * lane - j) << shift);
                            s_kk = kk - above;
                            break;
                        }
                        above += c[j];
                    }
                }
            }
            __syncthreads();
            prefix = s_prefix;
            kk = s_kk;
            mask |= 255u << shift;
        }
        T = prefix;
        need_eq = kk;
    }

    // ordered pass: token i is selected iff key > T, or key == T and fewer than need_eq equal keys precede it
    uint32_t G = 0, E = 0;           // selected-by-greater / equal counts before this chunk
    for (int c0 = 0; c0 < N_sel; c0 += kThreads * kItems) {
        const int base = c0 + tid * kItems;
        uint32_t gt[kItems], eq[kItems], tg = 0, te = 0;
#pragma unroll
        for (int u = 0; u < kItems; ++u) {
            int i = base + u;
            uint32_t key = (i < N_sel) ? score_key(s[i]) : 0u;
            gt[u] = (i < N_sel) && (key > T);
            eq[u] = (i < N_sel) && (key == T);
            tg += gt[u];
            te += eq[u];
        }
        uint32_t packed = tg | (te << 16);              // each count <= 4096 per chunk
        uint32_t inc = packed;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            uint32_t t = __shfl_up_sync(0xffffffffu, inc, o);
            if (lane >= o) inc += t;
        }
        if (lane == 31) warp_tot[warp] = inc;
        __syncthreads();
        if (warp == 0) {
            uint32_t w = warp_tot[lane], winc = w;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                uint32_t t = __shfl_up_sync(0xffffffffu, winc, o);
                if (lane >= o) winc += t;
            }
            warp_tot[lane] = winc - w;
            if (lane == 31) s_chunk_tot = winc;
        }
        __syncthreads();
        uint32_t exc = inc - packed + warp_tot[warp];
        uint32_t pg = G + (exc & 0xffffu), pe = E + (exc >> 16);
#pragma unroll
        for (int u = 0; u < kItems; ++u) {
            int i = base + u;
            if (i < N_sel) {
                bool take = gt[u] || (eq[u] && pe < need_eq);
                uint32_t before = pg + min(pe, need_eq);
                if (take) { if (sel) sel[before] = i; }
                else if (rem) rem[(uint32_t)i - before] = i;
                if (nsk) nsk[i] = take ? 0 : min(nsk[i] + 1, ASTRAEA_N_SKIP_CLAMP);
            }
            pg += gt[u];
            pe += eq[u];
        }
        uint32_t tot = s_chunk_tot;
        G += tot & 0xffffu;
        E += tot >> 16;
        __syncthreads();
    }
    for (int t = tid; t < n_always; t += kThreads) sel[k + t] = N_sel + t;
}

}  // namespace

size_t select_workspace_bytes(int, int) { return 256; }

int32_t launch_select(const float *score, int B, int N_sel, int k, int n_always, int32_t *idx_sel,
                      int32_t *idx_rem, int32_t *n_skip, void *, cudaStream_t stream)
{
    if (B == 0 || (N_sel == 0 && n_always == 0)) return ASTRAEA_OK;
    select_kernel<<<B, kThreads, 0, stream>>>(score, N_sel, k, n_always, idx_sel, idx_rem, n_skip);
    return check_launch("astraea_select");
}

}  // namespace astraea
