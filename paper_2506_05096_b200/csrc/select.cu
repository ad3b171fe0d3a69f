// astraea_select: budgeted top-k per batch row (Algorithm 1 line 3), deterministic.
//
// Scores are mapped to order-preserving 32-bit keys (larger score -> larger key; -0 == +0;
// NaN ranks as -inf).  A most-significant-digit radix select (4 passes of 8 bits, histogram
// in shared memory) finds the key T of the k-th largest score and how many scores equal to
// T still belong to the selection.  One ordered pass then writes both index lists in
// ascending token order with a block-wide prefix scan (no atomics on output positions), so
// equal scores go to the lower index, and updates the skip counters.
//
// Rows of up to 131072 tokens are handled by one thread-block cluster per batch row (up to 8 CTAs x 1024
// threads): every thread keeps its 2, 4, 8 or 16 consecutive keys in registers, so the scores are read from
// memory exactly once.  The digits are 12, 12 and 8 bits wide; per pass every CTA histograms its live keys in
// shared memory, adds its non-zero counts into EVERY CTA's copy of the cluster histogram with remote (DSMEM)
// atomics and, after one hardware cluster barrier, searches its own copy with all its threads.  The search
// stops as soon as the bin that holds the k-th key must be taken whole (float scores: after two passes, when
// the bin holds a single key); exact ties run all three passes.  The CTAs exchange their selected counts the
// same way to place their outputs.  Longer rows fall back to one CTA that re-reads the row from L2 in every
// pass (8-bit digits).  The call is latency-bound, not bandwidth-bound, at the sizes of the workloads, so the
// cluster kernel is launched with programmatic stream serialization: its CTAs become resident and clear their
// histograms while the kernel before them (the score kernel in a step) is still draining, and touch global
// memory only after griddepcontrol.wait.  (One CTA per row with the keys in shared memory was measured as
// well: 26.7 us on the 17550-token row against 16.7 us for a cluster of five, because one SM has to issue all
// of the ~100 instructions per token.)
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


// programmatic dependent launch: wait for the kernel before this one in the stream (all of its memory operations
// are then visible); let the kernel after this one start its own prologue
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// ---------------------------------------------------------------- cluster version (keys in registers)
constexpr int kMaxCluster = 8;
constexpr int kBinsWide = 4096;                  // 12-bit digits (the last digit has 8 bits and uses 256 of the bins)
constexpr int kPasses = 3;
constexpr size_t kClusterSmem = 2 * kPasses * kBinsWide * sizeof(uint32_t);      // own + cluster histogram per pass: 96 KB

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
    extern __shared__ __align__(16) uint32_t smem_hist[];      // [kPasses][kBinsWide] own counts, then [kPasses][kBinsWide] cluster counts
    uint32_t *hist = smem_hist, *ghist = smem_hist + kPasses * kBinsWide;
    __shared__ uint32_t cta_gt[kMaxCluster], cta_eq[kMaxCluster];   // selected-by-greater / equal totals of every CTA
    __shared__ uint32_t warp_tot[32], warp_gt[32], warp_eq[32];
    __shared__ uint32_t s_prefix, s_kk, s_cnt;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b = blockIdx.y;
    const uint32_t rank = cluster_rank(), csize = gridDim.x;
    const float *s = score + (size_t)b * N_sel;
    int32_t *sel = idx_sel ? idx_sel + (size_t)b * (k + n_always) : nullptr;
    int32_t *rem = idx_rem ? idx_rem + (size_t)b * (N_sel - k) : nullptr;
    int32_t *nsk = n_skip ? n_skip + (size_t)b * N_sel : nullptr;

    const int base = ((int)rank * kThreads + tid) * ITEMS;      // this thread's consecutive tokens
    {
        uint4 *z = reinterpret_cast<uint4 *>(smem_hist);
        for (int i = tid; i < (int)(kClusterSmem / 16); i += kThreads) z[i] = make_uint4(0, 0, 0, 0);
    }
    cluster_sync_all();                          // every CTA's histograms are zero before anyone adds to them (still ahead of the wait)
    grid_launch_dependents();                    // the next kernel may set itself up; it waits for this one before it reads anything
    grid_dependency_wait();                      // the scores (and whatever else the kernel before wrote) are complete
    uint32_t key[ITEMS];
    // the counters are needed only at the very end: fetched now where the registers allow it (16 items per thread
    // would spill), so that their latency is hidden behind the passes
    constexpr bool kPrefetchCounters = ITEMS <= 8;
    int32_t n_old[kPrefetchCounters ? ITEMS : 1];
    // a thread's tokens are consecutive: 16-byte accesses where the row's alignment and the thread's range allow them
    constexpr int kVec = ITEMS >= 4 ? 4 : ITEMS;
    const bool whole = base + ITEMS <= N_sel;
    const bool vec_s = whole && (reinterpret_cast<uintptr_t>(s + base) & (kVec * 4 - 1)) == 0;
    const bool vec_n = whole && nsk && (reinterpret_cast<uintptr_t>(nsk + base) & (kVec * 4 - 1)) == 0;
    if (vec_s) {
#pragma unroll
        for (int u = 0; u < ITEMS; u += kVec) {
            float f[kVec];
            if constexpr (kVec == 4) {
                const float4 v = __ldg(reinterpret_cast<const float4 *>(s + base + u));
                f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w;
            } else {
                const float2 v = __ldg(reinterpret_cast<const float2 *>(s + base + u));
                f[0] = v.x; f[1] = v.y;
            }
#pragma unroll
            for (int j = 0; j < kVec; ++j) key[u + j] = score_key(f[j]);
        }
    } else {
#pragma unroll
        for (int u = 0; u < ITEMS; ++u) key[u] = (base + u < N_sel) ? score_key(__ldg(s + base + u)) : 0u;
    }
    if constexpr (kPrefetchCounters) {
        if (vec_n) {
#pragma unroll
            for (int u = 0; u < ITEMS; u += kVec) {
                if constexpr (kVec == 4) {
                    const int4 v = *reinterpret_cast<const int4 *>(nsk + base + u);
                    n_old[u] = v.x; n_old[u + 1] = v.y; n_old[u + 2] = v.z; n_old[u + 3] = v.w;
                } else {
                    const int2 v = *reinterpret_cast<const int2 *>(nsk + base + u);
                    n_old[u] = v.x; n_old[u + 1] = v.y;
                }
            }
        } else {
#pragma unroll
            for (int u = 0; u < ITEMS; ++u) n_old[u] = (nsk && base + u < N_sel) ? nsk[base + u] : 0;
        }
    }

    // token i is selected iff key > T, or key == T and fewer than need_eq equal keys precede it
    uint32_t T = 0xffffffffu, need_eq = 0;       // no key reaches 0xffffffff
    if (k > 0) {
        uint32_t prefix = 0, mask = 0, kk = (uint32_t)k;
#pragma unroll 1
        for (int pass = 0; pass < kPasses; ++pass) {
            const int shift = pass == 0 ? 20 : pass == 1 ? 8 : 0;
            const uint32_t digit_mask = pass == 2 ? 255u : 4095u;
            uint32_t *h = hist + pass * kBinsWide, *gh = ghist + pass * kBinsWide;
#pragma unroll
            for (int u = 0; u < ITEMS; ++u) {
                const bool live = (base + u < N_sel) && ((key[u] & mask) == prefix);
                const uint32_t bin = (key[u] >> shift) & digit_mask;
                const uint32_t act = __ballot_sync(0xffffffffu, live);
                if (act == 0) continue;
                // the leading digits of the scores are nearly all equal: one atomic for the warp when its live keys
                // share the bin, else one per key (the later digits are spread out, so those rarely collide)
                const int leader = __ffs(act) - 1;
                const uint32_t lbin = __shfl_sync(0xffffffffu, bin, leader);
                if (__all_sync(0xffffffffu, !live || bin == lbin)) {
                    if (lane == leader) atomicAdd(&h[lbin], (uint32_t)__popc(act));
                } else if (live) {
                    atomicAdd(&h[bin], 1u);
                }
            }
            __syncthreads();
            // this CTA's non-zero counts go into every CTA's copy, so that every CTA searches its own copy
            const int bins = (int)digit_mask + 1;
            for (int i = tid; i < bins; i += kThreads) {
                const uint32_t c = h[i];
                if (c != 0)
                    for (uint32_t r = 0; r < csize; ++r) remote_add(map_to_rank(&gh[i], r), c);
            }
            cluster_sync_all();
            // search from the top: thread t owns bins top-4t .. top-4t-3 (the 256-bin pass uses the first 64 threads)
            {
                const int top = bins - 1 - 4 * tid;
                uint32_t c[4] = {0, 0, 0, 0}, tot = 0;
                if (top >= 3) {
#pragma unroll
                    for (int j = 0; j < 4; ++j) { c[j] = gh[top - j]; tot += c[j]; }
                }
                uint32_t inc = tot;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const uint32_t t = __shfl_up_sync(0xffffffffu, inc, o);
                    if (lane >= o) inc += t;
                }
                if (lane == 31) warp_tot[warp] = inc;
                __syncthreads();
                uint32_t wsum = warp_tot[lane];                  // every warp scans the 32 warp totals itself
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const uint32_t t = __shfl_up_sync(0xffffffffu, wsum, o);
                    if (lane >= o) wsum += t;
                }
                const uint32_t wbase = __shfl_sync(0xffffffffu, wsum, (warp + 31) & 31);
                const uint32_t exc = (warp > 0 ? wbase : 0u) + inc - tot;
                if (exc < kk && exc + tot >= kk) {
                    uint32_t above = exc;
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        if (above + c[j] >= kk) {
                            s_prefix = prefix | ((uint32_t)(top - j) << shift);
                            s_kk = kk - above;
                            s_cnt = c[j];
                            break;
                        }
                        above += c[j];
                    }
                }
                __syncthreads();
            }
            prefix = s_prefix;
            kk = s_kk;
            mask |= digit_mask << shift;
            if (s_cnt == kk) {
                // the whole bin is taken: every key with these leading digits is selected, whatever follows them
                T = prefix;                      // the smallest key of the bin, were it present
                need_eq = 0xffffffffu;
                break;
            }
            if (pass == kPasses - 1) { T = prefix; need_eq = kk; }
        }
    }

    // ordered placement
    uint32_t gtm = 0, eqm = 0;                   // bit u: this thread's token u has a key above / equal to T
#pragma unroll
    for (int u = 0; u < ITEMS; ++u) {
        const bool in = base + u < N_sel;
        gtm |= (uint32_t)(in && key[u] > T) << u;
        eqm |= (uint32_t)(in && key[u] == T) << u;
    }
    const uint32_t tg = __popc(gtm), te = __popc(eqm);
    uint32_t ig = tg, ie = te;                   // inclusive scans over the warp
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t a = __shfl_up_sync(0xffffffffu, ig, o), c = __shfl_up_sync(0xffffffffu, ie, o);
        if (lane >= o) { ig += a; ie += c; }
    }
    if (lane == 31) { warp_gt[warp] = ig; warp_eq[warp] = ie; }
    __syncthreads();
    uint32_t wg = warp_gt[lane], we = warp_eq[lane];            // every warp scans the 32 warp totals itself
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t a = __shfl_up_sync(0xffffffffu, wg, o), c = __shfl_up_sync(0xffffffffu, we, o);
        if (lane >= o) { wg += a; we += c; }
    }
    const uint32_t bg = warp > 0 ? __shfl_sync(0xffffffffu, wg, warp - 1) : 0u;
    const uint32_t be = warp > 0 ? __shfl_sync(0xffffffffu, we, warp - 1) : 0u;
    // every CTA learns every CTA's totals (the shuffles are outside the branch: all 32 lanes must take part)
    const uint32_t allg = __shfl_sync(0xffffffffu, wg, 31), alle = __shfl_sync(0xffffffffu, we, 31);
    if (warp == 0 && lane < (int)csize) {
        remote_store(map_to_rank(&cta_gt[rank], lane), allg);
        remote_store(map_to_rank(&cta_eq[rank], lane), alle);
    }
    cluster_sync_all();
    uint32_t pg = bg + ig - tg, pe = be + ie - te;
    for (uint32_t r = 0; r < rank; ++r) { pg += cta_gt[r]; pe += cta_eq[r]; }
    // With 8 or 16 tokens per thread a warp's direct stores of the two index lists would touch 32 lines per instruction
    // (a thread's entries are consecutive, the lanes are 32 or 64 bytes apart).  The warp's tokens are consecutive, and
    // so are their places in both lists: the entries are first put in order into the warp's piece of the histogram
    // memory (idle since the last cluster barrier; nobody writes it remotely any more), then copied out by whole lines.
    constexpr bool kStage = ITEMS >= 8;
    int32_t *stage = reinterpret_cast<int32_t *>(smem_hist) + warp * (32 * ITEMS);
    static_assert(!kStage || (size_t)kThreads * ITEMS * sizeof(int32_t) <= kClusterSmem, "the staged lists fit the histogram memory");
    const uint32_t before0 = pg + min(pe, need_eq);              // selected tokens ahead of this thread's first token
    const uint32_t takes = tg + min(te, need_eq > pe ? need_eq - pe : 0u);
    const uint32_t w_sel0 = __shfl_sync(0xffffffffu, before0, 0);
    const uint32_t w_sel_n = __shfl_sync(0xffffffffu, before0 + takes, 31) - w_sel0;     // selected tokens of the warp
    const int w_tok0 = base - lane * ITEMS;                      // the warp's first token
    const uint32_t w_rem0 = (uint32_t)w_tok0 - w_sel0;
#pragma unroll
    for (int u0 = 0; u0 < ITEMS; u0 += kVec) {
        int32_t cnt[kVec];                       // the counters of this group of tokens: old, then new
        if (vec_n) {
            if constexpr (kPrefetchCounters) {
#pragma unroll
                for (int j = 0; j < kVec; ++j) cnt[j] = n_old[u0 + j];
            } else if constexpr (kVec == 4) {    // not fetched ahead: one 16-byte load per four
                const int4 v = *reinterpret_cast<const int4 *>(nsk + base + u0);
                cnt[0] = v.x; cnt[1] = v.y; cnt[2] = v.z; cnt[3] = v.w;
            }
        }
#pragma unroll
        for (int j = 0; j < kVec; ++j) {
            const int u = u0 + j, i = base + u;
            if (i < N_sel) {
                const bool take = ((gtm >> u) & 1u) || (((eqm >> u) & 1u) && pe < need_eq);
                const uint32_t before = pg + min(pe, need_eq);
                if constexpr (kStage) {
                    if (take) stage[before - w_sel0] = i;
                    else stage[w_sel_n + ((uint32_t)i - before - w_rem0)] = i;
                } else {
                    if (take) { if (sel) sel[before] = i; }
                    else if (rem) rem[(uint32_t)i - before] = i;
                }
                if (vec_n) cnt[j] = take ? 0 : min(cnt[j] + 1, ASTRAEA_N_SKIP_CLAMP);
                else if (nsk) nsk[i] = take ? 0 : min((kPrefetchCounters ? n_old[u] : nsk[i]) + 1, ASTRAEA_N_SKIP_CLAMP);
            }
            pg += (gtm >> u) & 1u;
            pe += (eqm >> u) & 1u;
        }
        if (vec_n) {
            if constexpr (kVec == 4) *reinterpret_cast<int4 *>(nsk + base + u0) = make_int4(cnt[0], cnt[1], cnt[2], cnt[3]);
            else *reinterpret_cast<int2 *>(nsk + base + u0) = make_int2(cnt[0], cnt[1]);
        }
    }
    if constexpr (kStage) {
        __syncwarp();
        const int w_tok_n = min(max(N_sel - w_tok0, 0), 32 * ITEMS);      // tokens of this warp
        const uint32_t w_rem_n = (uint32_t)w_tok_n - w_sel_n;
        if (sel) for (uint32_t j = lane; j < w_sel_n; j += 32) sel[w_sel0 + j] = stage[j];
        if (rem) for (uint32_t j = lane; j < w_rem_n; j += 32) rem[w_rem0 + j] = stage[w_sel_n + j];
    }
    if (rank == 0) for (int t = tid; t < n_always; t += kThreads) sel[k + t] = N_sel + t;
    // no barrier at the end: the last remote accesses (the totals above) were complete at the barrier before the placement
}

template <int ITEMS>
int32_t launch_cluster(const float *score, int B, int N_sel, int k, int n_always, int32_t *idx_sel,
                       int32_t *idx_rem, int32_t *n_skip, cudaStream_t stream)
{
    const int csize = (N_sel + ITEMS * kThreads - 1) / (ITEMS * kThreads);
    static PerDeviceOnce attrs;                  // one per instantiation; the attribute is per device
    if (attrs.run([] { return cudaFuncSetAttribute(select_cluster_kernel<ITEMS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                   (int)kClusterSmem); }) != cudaSuccess)
        return check_launch("astraea_select (shared memory attribute)");
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(csize, B, 1);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = kClusterSmem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = csize;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;      // see grid_dependency_wait in the kernel
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
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
    if (N_sel > 0 && N_sel <= 2 * kThreads * kMaxCluster)
        return launch_cluster<2>(score, B, N_sel, k, n_always, idx_sel, idx_rem, n_skip, stream);
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
