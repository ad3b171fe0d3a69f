// astraea_select: budgeted top-k per batch row (Algorithm 1 line 3), deterministic.
//
// Scores are mapped to order-preserving 32-bit keys (larger score -> larger key; -0 == +0;
// NaN ranks as -inf).  A most-significant-digit radix select (4 passes of 8 bits, histogram
// in shared memory) finds the key T of the k-th largest score and how many scores equal to
// T still belong to the selection.  One ordered pass then writes both index lists in
// ascending token order with a block-wide prefix scan (no atomics on output positions), so
// equal scores go to the lower index, and updates the skip counters.
//
// Rows of up to 131072 tokens are handled by one thread-block cluster per batch row (up to 8
// CTAs x 1024 threads): every thread keeps its 4, 8 or 16 consecutive keys in registers, so the
// scores are read from memory exactly once; the per-CTA histograms are summed into the first CTA's
// shared memory with remote (DSMEM) atomics and every CTA searches the summed histogram itself; the
// CTAs exchange their selected counts the same way to place their outputs.  Cluster barriers are
// hardware barriers (no spinning).  Longer rows fall back to one CTA that re-reads the row from L2
// in every pass.  The call is latency-bound, not bandwidth-bound, at the sizes of the workloads.
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


// ---------------------------------------------------------------- cluster version (keys in registers)
constexpr int kMaxCluster = 8;

__device__ __forceinline__ uint32_t cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// address of the same shared-memory variable in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_rank(const void *p, uint32_t rank) {
    uint32_t a = static_cast<uint32_t>(__cvta_generic_to_shared(p)), r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(rank));
    return r;
}
__device__ __forceinline__ void remote_add(uint32_t addr, uint32_t v) {
    asm volatile("red.relaxed.cluster.shared::cluster.add.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
__device__ __forceinline__ void remote_store(uint32_t addr, uint32_t v) {
    asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}

template <int ITEMS>
__global__ void __launch_bounds__(kThreads)
select_cluster_kernel(const float *__restrict__ score, int N_sel, int k, int n_always,
                      int32_t *__restrict__ idx_sel, int32_t *__restrict__ idx_rem, int32_t *__restrict__ n_skip)
{
    __shared__ uint32_t hist[4][256];           // this CTA's histograms of the four passes
    __shared__ uint32_t ghist[4][256];          // the cluster's histograms: every CTA adds its counts into every CTA's copy
    __shared__ uint32_t cta_tot[kMaxCluster];   // packed (greater | equal << 16) totals of every CTA
    __shared__ uint32_t warp_tot[32];
    __shared__ uint32_t s_prefix, s_kk;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b = blockIdx.y;
    const uint32_t rank = cluster_rank(), csize = gridDim.x;
    const float *s = score + (size_t)b * N_sel;
    int32_t *sel = idx_sel ? idx_sel + (size_t)b * (k + n_always) : nullptr;
    int32_t *rem = idx_rem ? idx_rem + (size_t)b * (N_sel - k) : nullptr;
    int32_t *nsk = n_skip ? n_skip + (size_t)b * N_sel : nullptr;

    const int base = ((int)rank * kThreads + tid) * ITEMS;      // this thread's consecutive tokens
    uint32_t key[ITEMS];
#pragma unroll
    for (int u = 0; u < ITEMS; ++u) key[u] = (base + u < N_sel) ? score_key(__ldg(s + base + u)) : 0u;

    for (int i = tid; i < 4 * 256; i += kThreads) { (&ghist[0][0])[i] = 0; (&hist[0][0])[i] = 0; }
    cluster_sync_all();                          // every CTA's histograms are zero before anyone adds to them

    uint32_t T = 0xffffffffu, need_eq = 0;       // no key reaches 0xffffffff
    if (k > 0) {
        uint32_t prefix = 0, mask = 0, kk = (uint32_t)k;
#pragma unroll 1
        for (int pass = 0; pass < 4; ++pass) {
            const int shift = 24 - 8 * pass;
#pragma unroll
            for (int u = 0; u < ITEMS; ++u) {
                const bool live = (base + u < N_sel) && ((key[u] & mask) == prefix);
                const uint32_t bin = (key[u] >> shift) & 255u;
                const uint32_t act = __ballot_sync(0xffffffffu, live);
                if (act == 0) continue;
                // the leading digits of the scores are nearly all equal: one atomic for the warp when its live keys
                // share the bin, else one per key (the later digits are spread out, so those rarely collide)
                const int leader = __ffs(act) - 1;
                const uint32_t lbin = __shfl_sync(0xffffffffu, bin, leader);
                if (__all_sync(0xffffffffu, !live || bin == lbin)) {
                    if (lane == leader) atomicAdd(&hist[pass][lbin], (uint32_t)__popc(act));
                } else if (live) {
                    atomicAdd(&hist[pass][bin], 1u);
                }
            }
            __syncthreads();
            // thread (r, bin) adds this CTA's count of the bin into CTA r's copy, so that every CTA searches its own copy
            for (int i = tid; i < 256 * (int)csize; i += kThreads) {
                const uint32_t c = hist[pass][i & 255];
                if (c != 0) remote_add(map_to_rank(&ghist[pass][i & 255], (uint32_t)i >> 8), c);
            }
            cluster_sync_all();
            if (warp == 0) {
                // lane l owns bins 255-8l .. 248-8l (descending); find where the count from the top reaches kk
                uint32_t c[8], tot = 0;
#pragma unroll
                for (int j = 0; j < 8; ++j) { c[j] = ghist[pass][255 - 8 * lane - j]; tot += c[j]; }
                uint32_t inc = tot;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    uint32_t t = __shfl_up_sync(0xffffffffu, inc, o);
                    if (lane >= o) inc += t;
                }
                const uint32_t exc = inc - tot;
                if (exc < kk && inc >= kk) {
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

    // ordered placement: token i is selected iff key > T, or key == T and fewer than need_eq equal keys precede it
    uint32_t gt[ITEMS], eq[ITEMS], tg = 0, te = 0;
#pragma unroll
    for (int u = 0; u < ITEMS; ++u) {
        const bool in = base + u < N_sel;
        gt[u] = in && key[u] > T;
        eq[u] = in && key[u] == T;
        tg += gt[u];
        te += eq[u];
    }
    const uint32_t packed = tg | (te << 16);     // a CTA holds at most 16384 tokens
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
        // every CTA learns every CTA's totals
        const uint32_t total = __shfl_sync(0xffffffffu, winc, 31);
        if (lane < csize) remote_store(map_to_rank(&cta_tot[rank], lane), total);
    }
    cluster_sync_all();
    uint32_t G = 0, E = 0;
    for (uint32_t r = 0; r < rank; ++r) { G += cta_tot[r] & 0xffffu; E += cta_tot[r] >> 16; }
    const uint32_t exc = inc - packed + warp_tot[warp];
    uint32_t pg = G + (exc & 0xffffu), pe = E + (exc >> 16);
#pragma unroll
    for (int u = 0; u < ITEMS; ++u) {
        const int i = base + u;
        if (i < N_sel) {
            const bool take = gt[u] || (eq[u] && pe < need_eq);
            const uint32_t before = pg + min(pe, need_eq);
            if (take) { if (sel) sel[before] = i; }
            else if (rem) rem[(uint32_t)i - before] = i;
            if (nsk) nsk[i] = take ? 0 : min(nsk[i] + 1, ASTRAEA_N_SKIP_CLAMP);
        }
        pg += gt[u];
        pe += eq[u];
    }
    if (rank == 0) for (int t = tid; t < n_always; t += kThreads) sel[k + t] = N_sel + t;
    // no barrier at the end: the last remote accesses (the totals above) were complete at the barrier before the placement
}

template <int ITEMS>
int32_t launch_cluster(const float *score, int B, int N_sel, int k, int n_always, int32_t *idx_sel,
                       int32_t *idx_rem, int32_t *n_skip, cudaStream_t stream)
{
    const int csize = (N_sel + ITEMS * kThreads - 1) / (ITEMS * kThreads);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(csize, B, 1);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = csize;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, select_cluster_kernel<ITEMS>, score, N_sel, k, n_always, idx_sel, idx_rem, n_skip);
    if (e != cudaSuccess) return fail(ASTRAEA_ERR_CUDA, "astraea_select: %s", cudaGetErrorString(e));
    return check_launch("astraea_select");
}

}  // namespace

size_t select_workspace_bytes(int, int) { return 256; }

int32_t launch_select(const float *score, int B, int N_sel, int k, int n_always, int32_t *idx_sel,
                      int32_t *idx_rem, int32_t *n_skip, void *, cudaStream_t stream)
{
    if (B == 0 || (N_sel == 0 && n_always == 0)) return ASTRAEA_OK;
#ifdef SEL_FORCE
    if (N_sel > 0 && N_sel <= SEL_FORCE * kThreads * kMaxCluster) return launch_cluster<SEL_FORCE>(score, B, N_sel, k, n_always, idx_sel, idx_rem, n_skip, stream);
#endif
    if (N_sel > 0 && N_sel <= 4 * kThreads * kMaxCluster)
        return launch_cluster<4>(score, B, N_sel, k, n_always, idx_sel, idx_rem, n_skip, stream);
    if (N_sel > 0 && N_sel <= 8 * kThreads * kMaxCluster)
        return launch_cluster<8>(score, B, N_sel, k, n_always, idx_sel, idx_rem, n_skip, stream);
    if (N_sel > 0 && N_sel <= 16 * kThreads * kMaxCluster)
        return launch_cluster<16>(score, B, N_sel, k, n_always, idx_sel, idx_rem, n_skip, stream);
    select_kernel<<<B, kThreads, 0, stream>>>(score, N_sel, k, n_always, idx_sel, idx_rem, n_skip);
    return check_launch("astraea_select");
}

}  // namespace astraea
