// astraea_sparse_attn: out[i] = Softmax(q_i K^T * scale) V for the selected query rows i
// against ALL keys/values, written in place over the cached output (Algorithm 1 lines 6-7;
// Section 3.2 "Sparse Attention").
//
// One CTA per (256 selected queries, head, batch): two 128-row query tiles that share every
// K/V tile of 64 keys.  (The CTAs of a launch's last, partial round may instead be replaced by several CTAs
// each, every one with a share of the key tiles; merge_parts_kernel combines their rows: see SplitPlan.)  Warp roles:
//   softmax warpgroups (one thread per query row), two per query tile: gather the tile's Q rows into
//              128B-swizzled shared memory, then per key tile read S from TMEM, exponentiate in the log2
//              domain against a reference maximum, write P (bf16) back to TMEM over S, and at the end
//              normalise O and scatter it to the rows q_idx names;
//   one warp   TMA producer: K and V tiles into multi-stage swizzled buffers;
//   two warps  tcgen05.mma issuers, one per query tile: S = Q K^T (SS, K-major operands), O += P V (P from
//              TMEM, V as an MN-major shared-memory operand); the first owns the TMEM allocation;
//   one warp   only donates registers (setmaxnreg moves registers to the softmax warps).
//
// Two softmax warpgroups per query tile put four softmax warps on every SM sub-partition, which hides the
// serial chain of a key tile (wait, load, exponentials, sum, pack, publish).  Even key tiles go to one
// warpgroup and odd ones to the other, each with an S buffer of its own, which is refilled with key tile
// j+2 as soon as P of tile j has been consumed (the tensor pipe executes one thread's MMAs in order); both
// work against the same reference maximum and their P tiles accumulate into ONE O accumulator per query
// tile.
//
// The softmax is bound by the exponentials (XU pipe, 16 per clock per SM), by the issue slots and by the
// latencies of its own chain, so the common path of a key tile is kept to: load S, one FFMA + one
// exponential per element, (sum,) pack, store.  At head_dim 64 / 72 six / four of every sixteen
// exponentials are a cubic on the FMA pipe instead of ex2 on the XU, and at head_dim 64 the row sums are
// left to the tensor core (P times a column of ones, 16 more accumulator columns).  The reference maximum
// is the exact row maximum of key tile 0 (plus a shift) and is then only checked through the sums of
// exponentials: while they stay below a limit the probabilities are accepted as they are (they are relative
// to a stale maximum, which the final normalisation cancels; fp32 and bf16 have the range).  Otherwise the
// CTA raises a flag, finishes the pass, and redoes its work in two more passes over the keys: exact row
// maxima first, then the softmax against them (the accumulator is shared by two warpgroups, so it is not
// rescaled in place).
//
// At head_dim 64 / 72 the kernel also exists with ONE query tile per CTA and two CTAs per SM (half the TMEM, at
// most 113 KB of shared memory each): per SM that is 5-17 % slower, but its CTAs are half as long, so a launch of
// only a few rounds of CTAs finishes earlier with it; the launch estimates both and picks.
//
// TMEM columns: S/P of (tile t, buffer u) at (kSBufs t + u) * kBlockN; the O accumulators behind them.
// The producer and issuer warps run warp-uniform code and elect one lane per instruction, so
// that descriptors and addresses stay in uniform registers (a lone diverged thread issues
// tcgen05.mma several times slower).  Every mbarrier wait is bounded; on a timeout the CTA raises
// the error word, the remaining waits return at once, and the CTA runs out.
#include <mutex>

#include "common.cuh"
#include "sm100_ptx.cuh"
#include "bounded_wait.cuh"

namespace astraea {
namespace {

using namespace ptx;

constexpr int kBlockM = 128;                     // rows of one query tile
constexpr int kSplit = 2;                        // softmax warpgroups per query tile: one takes the even key tiles, one the odd
// The speculative reference of a row is the exact maximum of its first key tile plus kRefShift (log2 domain), and
// a tile whose sum of exponentials passes kTileSumLimit means that this reference is too low.  fp32 and bf16 share
// the exponent range and keep their relative precision across it, so the reference may sit anywhere in a wide
// window: the shift leaves 2^-48 .. 2^-126 for the terms below a maximum that IS in the first tile (78 bits), and
// the limit leaves 2^27 of head room above 2^100 for the number of keys times the magnitude of the values.
// Together a later key may beat the first tile's maximum by 148 * ln 2 = 102 nats before the CTA has to redo its
// work, which costs two more passes over the keys: heavy-tailed logits (per-token norms) reach 40-60 nats in some
// row of most CTAs, but not 100.
constexpr float kRefShift = 48.0f;
constexpr float kTileSumLimit = 1267650600228229401496703205376.0f;   // 2^100

// DH: head_dim.  TM: 128-row query tiles per CTA.  Two share every K/V tile in shared memory and run one CTA per SM;
// one (head_dim 64 / 72 only) lets two CTAs share an SM, which costs ~5 % of throughput per SM but halves the
// granularity of the schedule: launches of only a few rounds of CTAs are faster with it.
template <int DH, int TM> struct Cfg {
    static constexpr int kDH = DH;
    static constexpr int kTilesM = TM;
    static constexpr int kCtasPerSM = (TM == 1) ? 2 : 1;
    static constexpr uint32_t kTmemCols = 512 / kCtasPerSM;
    static_assert(TM == 2 || DH != 128, "head_dim 128 needs the whole SM");
    // head_dim = kMain (whole 64-column, 128-byte-swizzled chunks) + kTail (8 columns at head_dim 72,
    // carried as a 16-column, 32-byte-swizzled chunk whose upper half is zero)
    static constexpr int kMain = DH / 64 * 64;
    static constexpr int kTail = DH - kMain;
    static constexpr int kTailPad = kTail ? 16 : 0;
    static_assert(kTail == 0 || kTail == 8, "head_dim must be 64, 72 or 128");
    static constexpr int kBlockN = 64;                            // keys per K/V tile = columns of an S buffer
    // Row sums by the tensor core at head_dim 64: P times a column of ones into 16 more accumulator columns.  That
    // takes the 64 packed adds per key tile off the softmax warps, whose issue slots are what is short there
    // (+6 %), and normalises O by the sum of the very bf16 probabilities that went into it; the row sum, and with it
    // the LSE, then carries the bf16 rounding of the probabilities (up to 2^-8 relative when one key dominates a row).
    // head_dim 72 gains nothing from it and 128 has no TMEM columns left: they sum the fp32 exponentials themselves.
    static constexpr bool kOnes = DH == 64;
    static constexpr int kSBufs = 2;                              // S buffers per query tile: one per softmax warpgroup
    // exponentials per 16 that are computed on the FMA pipe instead of the XU (measured best: 6 at head_dim 64, 4 at
    // 72, none at 128, where the tensor pipe is as busy as the XU)
    static constexpr int kPolyOf16 = (DH == 64) ? 6 : (DH == 72) ? 4 : 0;
    static constexpr int kSoftmaxWarps = 4 * kTilesM * kSplit;
    static constexpr int kAhead = kSBufs;                         // Q K^T runs this many key tiles ahead of P V
    static constexpr int kThreads = (kSoftmaxWarps + 4) * 32;     // + producer, two issuers, one register donor
    static constexpr uint32_t kColO = kTilesM * kSBufs * kBlockN; // first O column
    static constexpr uint32_t kOnesCol = kMain + kTailPad;       // accumulator column that receives the row sums
    static constexpr uint32_t kOStride = kMain + kTailPad + (kOnes ? 16 : 0);   // columns between O accumulators
    static_assert(kColO + kTilesM * kOStride <= kTmemCols, "TMEM budget");
    // setmaxnreg only redistributes what the CTA got at launch: an increase that the decreases of
    // the last warpgroup cannot cover would block forever
    static constexpr int kRegsLaunch = (65536 / kCtasPerSM / kThreads) / 8 * 8;
    static constexpr int kRegsSoftmax = (kCtasPerSM == 2) ? 104 : 112, kRegsOther = 32;
    static_assert(kRegsSoftmax * kSoftmaxWarps * 32 + kRegsOther * 128 <= kRegsLaunch * kThreads, "setmaxnreg budget");
    static constexpr int kChunks = kMain / 64;                    // 64-column (128-byte) swizzle chunks
    static constexpr int kQChunkBytes = kBlockM * 128;            // 128 query rows x 128 bytes
    static constexpr int kQTailBytes = kTail ? kBlockM * 32 : 0;  // 128 query rows x 32 bytes
    static constexpr int kQTileBytes = kChunks * kQChunkBytes + kQTailBytes;
    static constexpr int kChunkBytes = kBlockN * 128;             // one key tile x 128 bytes
    static constexpr int kTailBytes = kTail ? kBlockN * 32 : 0;   // one key tile x 32 bytes
    static constexpr int kLoadBytes = kChunks * kChunkBytes + kTailBytes;   // what TMA delivers per K or V tile
    static constexpr int kTileBytes = (kLoadBytes + 1023) / 1024 * 1024;    // stage size (keeps the swizzle alignment)
    static_assert(kQTileBytes % 1024 == 0 && kTileBytes % 1024 == 0, "tiles keep the 1024-byte swizzle alignment");
    static constexpr int kStagesK = (kCtasPerSM == 2) ? 4 : (DH == 128) ? 5 : 6;     // two CTAs per SM: <= 113 KB each
    static constexpr int kStagesV = (kCtasPerSM == 2) ? 4 : (DH == 128) ? 4 : 6;
    static_assert(kStagesK > kAhead, "K runs kAhead tiles ahead");
    static constexpr int kBarBytes = 512;
    static constexpr int kOnesBytes = kOnes ? kBlockN * 32 : 0;  // a key tile x 16 columns of bf16: ones in column 0
    static constexpr int kSmemBytes = kQTileBytes * kTilesM + kTileBytes * (kStagesK + kStagesV) + kOnesBytes + kBarBytes + 1024;
};

struct Params {
    const __nv_bfloat16 *q;
    int64_t q_sb, q_sh, q_sn;
    const int32_t *q_idx;
    int M;
    __nv_bfloat16 *out;
    float *lse_out;
    int N, H;                    // N: keys
    int N_tok;                   // tokens of q / out / lse_out (N_tok == N unless the keys were gathered)
    float scale, scale_log2;
    int compact;
    int h0;                      // first head of this launch
    int *err_word;
    // The grid is one-dimensional: CTA id -> (query-tile group x, head y, batch z), x fastest.  CTAs [0, n_full) take
    // their rows against all keys.  Every later group of `split` CTAs shares one such unit and splits its KEY tiles
    // evenly: each writes normalised fp32 rows and their LSE to part_o / part_lse, which merge_parts_kernel combines.
    int tiles_x, heads;
    int n_full, split;
    float *part_o, *part_lse;    // [part][kTilesM * 128 rows][head_dim] and [part][kTilesM * 128 rows]
};

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// packed fp32 pairs: one issue slot for two FMAs / adds
__device__ __forceinline__ void ffma2(float &x0, float &x1, float m, float c) {
    unsigned long long a, b, d, r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(a) : "f"(x0), "f"(x1));
    asm("mov.b64 %0, {%1, %1};" : "=l"(b) : "f"(m));
    asm("mov.b64 %0, {%1, %1};" : "=l"(d) : "f"(c));
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(d));
    asm("mov.b64 {%0, %1}, %2;" : "=f"(x0), "=f"(x1) : "l"(r));
}
__device__ __forceinline__ unsigned long long fadd2(unsigned long long a, float x0, float x1) {
    unsigned long long b, r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(b) : "f"(x0), "f"(x1));
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}

// 2^x for a pair, without the XU pipe: x = n + f with n = floor(x) taken by adding 1.5 * 2^23 rounded down, a
// cubic for 2^f on [0, 1) (relative error 8.6e-5, well below the bf16 rounding of P), and n added to the
// exponent field.  x is clamped to the normal range first: below it the result is 2^-126 instead of 0, which no sum
// notices; above it the exponent field would wrap around to a small number and hide the overflow from the check
// on the tile's sum, so x stops at 127, whose 2^127 trips that check as surely as the XU's +inf does.
__device__ __forceinline__ void exp2_poly2(float &x0, float &x1) {
    x0 = fminf(fmaxf(x0, -126.0f), 127.0f);
    x1 = fminf(fmaxf(x1, -126.0f), 127.0f);
    unsigned long long x, t, pl;
    asm("mov.b64 %0, {%1, %2};" : "=l"(x) : "f"(x0), "f"(x1));
    asm("{\n\t.reg .b64 mg, c1, c2, c3, one, fr;\n\t"
        "mov.b64 mg, 0x4B4000004B400000;\n\t"        // 1.5 * 2^23, twice
        "mov.b64 c3, 0x3D9DD4DF3D9DD4DF;\n\t"        // 2^f ~ 1 + f (c1 + f (c2 + f c3))
        "mov.b64 c2, 0x3E691C043E691C04;\n\t"
        "mov.b64 c1, 0x3F31F3293F31F329;\n\t"
        "mov.b64 one, 0x3F8000003F800000;\n\t"
        "add.rm.f32x2 %0, %2, mg;\n\t"               // low mantissa bits of t = floor(x)
        "sub.rn.f32x2 fr, %0, mg;\n\t"
        "sub.rn.f32x2 fr, %2, fr;\n\t"               // f = x - floor(x)
        "fma.rn.f32x2 %1, fr, c3, c2;\n\t"
        "fma.rn.f32x2 %1, %1, fr, c1;\n\t"
        "fma.rn.f32x2 %1, %1, fr, one;\n\t}"
        : "=&l"(t), "=&l"(pl) : "l"(x));
    uint32_t t0, t1, p0, p1;
    asm("mov.b64 {%0, %1}, %2;" : "=r"(t0), "=r"(t1) : "l"(t));
    asm("mov.b64 {%0, %1}, %2;" : "=r"(p0), "=r"(p1) : "l"(pl));
    x0 = __uint_as_float(p0 + (t0 << 23));
    x1 = __uint_as_float(p1 + (t1 << 23));
}

__device__ __forceinline__ float max3(float a, float b, float c) {
    float r;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}

struct Bars {
    uint32_t q;                     // [kTilesM]
    uint32_t s, p;                  // [kTilesM][4]: one per S buffer (S is there; P is there)
    uint32_t done;                  // [kTilesM]: every P V of the pass has landed
    uint32_t kf, ke, vf, ve;        // [stages]
};

struct SoftmaxState {
    float sl2, m_ref, l_sum;
    float shift;                    // the exponentials are taken against m_ref * sl2 + shift (log2 domain)
    uint32_t t_s0, t_o, bar_s, bar_p, bar_done;
    int N;                          // keys
    float *ref_x;                   // the reference of this thread's row, shared by the tile's two warpgroups
    int ref_bar;                    // named barrier on which the reference is handed over
    volatile int *redo_flag;
    volatile int *abort_flag;
    int *err_word;
};

// the 64 columns of one S buffer into registers (asynchronous: wait_s_regs before using them)
template <int NS>
__device__ __forceinline__ void load_s(uint32_t t_s, float (&s)[NS]) {
    static_assert(NS == 64, "an S buffer has 64 columns");
    tmem_ld32(t_s, reinterpret_cast<uint32_t (&)[32]>(s[0]));
    tmem_ld32(t_s + 32, reinterpret_cast<uint32_t (&)[32]>(s[32]));
}
// tcgen05.wait::ld that names the loaded registers, so that no use of them can move above it
__device__ __forceinline__ void wait_regs16(float *s) {
    asm volatile("tcgen05.wait::ld.sync.aligned;"
        : "+f"(s[0]), "+f"(s[1]), "+f"(s[2]), "+f"(s[3]), "+f"(s[4]), "+f"(s[5]), "+f"(s[6]), "+f"(s[7]),
          "+f"(s[8]), "+f"(s[9]), "+f"(s[10]), "+f"(s[11]), "+f"(s[12]), "+f"(s[13]), "+f"(s[14]), "+f"(s[15])
        :: "memory");
}
template <int NS>
__device__ __forceinline__ void wait_s_regs(float (&s)[NS]) {
    static_assert(NS % 16 == 0, "sixteen registers per wait");
#pragma unroll
    for (int i = 0; i < NS; i += 16) wait_regs16(&s[i]);      // waits after the first are free; they only tie registers
}

// keys beyond `valid` (zero-filled tail of the last key tile) get logit -inf
template <int NS>
__device__ __forceinline__ void mask_tail(float (&s)[NS], int valid) {
    if (valid < NS) {
#pragma unroll
        for (int i = 0; i < NS; ++i) if (i >= valid) s[i] = -INFINITY;
    }
}

template <int NS>
__device__ __forceinline__ float row_max(const float (&s)[NS]) {
    float mx4[4] = {max3(s[0], s[1], s[2]), max3(s[3], s[4], s[5]), max3(s[6], s[7], s[8]), max3(s[9], s[10], s[11])};
#pragma unroll
    for (int i = 12; i + 7 < NS; i += 8) {
        mx4[0] = max3(mx4[0], s[i], s[i + 1]); mx4[1] = max3(mx4[1], s[i + 2], s[i + 3]);
        mx4[2] = max3(mx4[2], s[i + 4], s[i + 5]); mx4[3] = max3(mx4[3], s[i + 6], s[i + 7]);
    }
    static_assert((NS - 12) % 8 == 4, "tail of the max tree");
    mx4[0] = max3(mx4[0], s[NS - 4], s[NS - 3]);
    mx4[1] = max3(mx4[1], s[NS - 2], s[NS - 1]);
    return fmaxf(max3(mx4[0], mx4[1], mx4[2]), mx4[3]);
}

template <int NS>
__device__ __forceinline__ void pack_p(const float (&e)[NS], uint32_t (&pk)[NS / 2]) {
#pragma unroll
    for (int i = 0; i < NS / 2; ++i) {
        __nv_bfloat162 v2 = __floats2bfloat162_rn(e[2 * i], e[2 * i + 1]);
        pk[i] = *reinterpret_cast<uint32_t *>(&v2);
    }
}

// P of one key tile: NS/2 packed bf16 pairs over the first NS/2 columns of the S buffer
template <int NS>
__device__ __forceinline__ void store_p(uint32_t t_s, const uint32_t (&pk)[NS / 2]) {
    static_assert(NS == 64, "an S buffer has 64 columns");
    tmem_st32(t_s, pk);
}

// P has been stored: make it visible to the issuer warp
__device__ __forceinline__ void publish_p(uint32_t bar) {
    tc_wait_st();
    tc_fence_before();
    mbar_arrive(bar);
}

// What a pass over the keys does (only kSpeculate unless a tile overflowed):
//   kSpeculate  exponentials against the exact row maximum of key tile 0; a tile whose sum of exponentials passes
//               the limit raises the CTA's redo flag (the accumulator is shared by two warpgroups, so nothing
//               is repaired in place);
//   kMaxOnly    first pass of a redo: only the exact row maxima over all keys are taken;
//   kExact      second pass of a redo: exponentials against those maxima, nothing can overflow.
enum { kSpeculate = 0, kMaxOnly = 1, kExact = 2 };

// One key tile of the softmax.  j: key tile; g: running count of S-buffer uses of this query tile (buffer
// g % kSBufs, barrier phase (g / kSBufs) & 1), which keeps counting across the passes.
template <class C, int MODE>
__device__ __forceinline__ void softmax_step(SoftmaxState &st, int j, int g)
{
    constexpr int kSBufs = C::kSBufs, NS = C::kBlockN;
    const int buf = g % kSBufs;
    const uint32_t t_s = st.t_s0 + buf * NS;
    const float sl2 = st.sl2;
    float cur[NS];
    // the load is waited for at once: registers of a tcgen05.ld in flight must not be touched, and the
    // compiler cannot know that
    wait_bar(st.bar_s + 8 * buf, (g / kSBufs) & 1, st.abort_flag, st.err_word);
    tc_fence_after();
    load_s<NS>(t_s, cur);
    wait_s_regs<NS>(cur);
    mask_tail<NS>(cur, st.N - j * NS);
    if constexpr (MODE == kMaxOnly) {
        st.m_ref = fmaxf(st.m_ref, row_max<NS>(cur));
        tc_fence_before();
        mbar_arrive(st.bar_p + 8 * buf);              // S has been read: the buffer may be refilled
        return;
    }
    if (MODE == kSpeculate && j == 0) {
        // the reference is the exact maximum of the first key tile; the other warpgroup of this query tile takes the same one
        st.m_ref = row_max<NS>(cur);
        *st.ref_x = st.m_ref;
        if (st.ref_bar == 3) asm volatile("bar.arrive 3, 256;" ::: "memory");
        else asm volatile("bar.arrive 4, 256;" ::: "memory");
    }
    const float neg = -st.m_ref * sl2 - st.shift;
#pragma unroll
    for (int i = 0; i < NS; i += 2) ffma2(cur[i], cur[i + 1], sl2, neg);
    // kPolyOf16 of every 16 exponentials go to the FMA pipe, the rest to the XU
#pragma unroll
    for (int i = 0; i < NS; i += 16) {
#pragma unroll
        for (int u = 0; u < 16; u += 2) {
            if (u >= 16 - C::kPolyOf16) exp2_poly2(cur[i + u], cur[i + u + 1]);
            else { cur[i + u] = ex2(cur[i + u]); cur[i + u + 1] = ex2(cur[i + u + 1]); }
        }
    }
    float tile_sum = 0.f;
    if constexpr (!C::kOnes) {
        unsigned long long a[4] = {0ull, 0ull, 0ull, 0ull};
#pragma unroll
        for (int i = 0; i < NS; i += 8) {
#pragma unroll
            for (int u = 0; u < 4; ++u) a[u] = fadd2(a[u], cur[i + 2 * u], cur[i + 2 * u + 1]);
        }
        float f[8];
#pragma unroll
        for (int u = 0; u < 4; ++u) asm("mov.b64 {%0, %1}, %2;" : "=f"(f[2 * u]), "=f"(f[2 * u + 1]) : "l"(a[u]));
        tile_sum = ((f[0] + f[1]) + (f[2] + f[3])) + ((f[4] + f[5]) + (f[6] + f[7]));
    }
    // P as bf16 pairs (element 2c in the low half); packed before the check below so that the conversions run
    // in the shadow of the sum and the vote
    uint32_t pk[NS / 2];
    pack_p<NS>(cur, pk);
    if constexpr (MODE == kSpeculate && !C::kOnes) {
        // rare: the reference is too low for this tile.  The CTA finishes the pass and redoes its work with exact maxima
        if (__any_sync(0xffffffffu, !(tile_sum <= kTileSumLimit))) *st.redo_flag = 1;
    }
    st.l_sum += tile_sum;
    store_p<NS>(t_s, pk);                         // over the first NS/2 columns of this S buffer
    publish_p(st.bar_p + 8 * buf);
}

// All warps of the CTA meet after the speculative pass and then agree on the redo flag.
template <class C>
__device__ __forceinline__ void pass_sync() {
    asm volatile("bar.sync 5, %0;" ::"n"(C::kThreads) : "memory");
}

// ---------------------------------------------------------------- softmax warpgroup
// tile: its query tile; par: which key tiles it takes (j = par, par + kSplit, ...)
template <class C>
__device__ __forceinline__ void softmax_role(const Params &p, const Bars &bar, int tile, int par, uint8_t *sQ_gen, uint32_t tmem,
                                             int m_base, int h, int b, int n_tiles, int key0, int part,
                                             volatile int *abort_flag, volatile int *redo_flag, float2 *xchg)
{
    const int wtid = threadIdx.x & 127;
    const int warp = __shfl_sync(0xffffffffu, wtid >> 5, 0);       // warp-uniform
    // gather this tile's Q rows (swizzled, K-major): 16-byte units, unit c of row r
    constexpr int kMainUnits = C::kMain / 8, kUnits = kMainUnits + (C::kTail ? 2 : 0);
    // (the warpgroups of a tile share the rows; all index loads first, then all row loads, then the stores, so that the
    // two dependent round trips to memory are paid once and not once per unit)
    constexpr int kGatherIters = kBlockM * kUnits / (128 * kSplit);
    static_assert(kBlockM * kUnits % (128 * kSplit) == 0, "whole iterations of the Q gather");
    int gtok[kGatherIters];
#pragma unroll
    for (int it = 0; it < kGatherIters; ++it) {
        const int v = par * 128 + wtid + it * 128 * kSplit;
        const int r = v / kUnits, c = v - r * kUnits;
        const int m = m_base + r;
        gtok[it] = -1;
        if (m < p.M && c * 8 < C::kDH)                   // the upper half of the tail chunk stays zero
            gtok[it] = p.q_idx ? __ldg(p.q_idx + (size_t)b * p.M + m) : m;
    }
    uint4 gval[kGatherIters];
#pragma unroll
    for (int it = 0; it < kGatherIters; ++it) {
        const int v = par * 128 + wtid + it * 128 * kSplit;
        const int c = v % kUnits;
        gval[it] = make_uint4(0, 0, 0, 0);
        if ((unsigned)gtok[it] < (unsigned)p.N_tok) {
            const __nv_bfloat16 *src = p.q + (size_t)b * p.q_sb + (size_t)gtok[it] * p.q_sn + (size_t)h * p.q_sh + c * 8;
            gval[it] = __ldg(reinterpret_cast<const uint4 *>(src));
        }
    }
#pragma unroll
    for (int it = 0; it < kGatherIters; ++it) {
        const int v = par * 128 + wtid + it * 128 * kSplit;
        const int r = v / kUnits, c = v - r * kUnits;
        uint32_t off;
        if (c < kMainUnits) off = (c >> 3) * C::kQChunkBytes + r * 128 + (((c & 7) ^ (r & 7)) << 4);          // 128-byte swizzle
        else off = C::kChunks * C::kQChunkBytes + r * 32 + ((((c - kMainUnits) & 1) ^ ((r >> 2) & 1)) << 4);   // 32-byte swizzle
        *reinterpret_cast<uint4 *>(sQ_gen + off) = gval[it];
    }
    fence_proxy_async_smem();
    mbar_arrive(bar.q + 8 * tile);

    const uint32_t t_row = tmem + ((uint32_t)(warp * 32) << 16);
    SoftmaxState st;
    st.sl2 = p.scale_log2;
    st.l_sum = 0.f;
    st.t_s0 = t_row + tile * C::kSBufs * C::kBlockN;
    st.t_o = t_row + C::kColO + tile * C::kOStride;
    st.bar_s = bar.s + 32 * tile; st.bar_p = bar.p + 32 * tile; st.bar_done = bar.done + 8 * tile;
    st.N = p.N - key0;                                           // keys from this CTA's first key tile on
    st.abort_flag = abort_flag; st.err_word = p.err_word;
    st.ref_x = &xchg[wtid].x; st.ref_bar = 3 + tile; st.redo_flag = redo_flag;

    const int m = m_base + wtid;
    int tok = -1;
    if (m < p.M) {
        tok = p.q_idx ? __ldg(p.q_idx + (size_t)b * p.M + m) : m;
        // an entry out of range, or one that does not exceed its predecessor (two rows would race on one output
        // row), is reported and its row is not written
        const bool bad = (unsigned)tok >= (unsigned)p.N_tok ||
                         (p.q_idx && m > 0 && __ldg(p.q_idx + (size_t)b * p.M + m - 1) >= tok);
        if (bad) { if (par == 0 && p.err_word) atomicExch(p.err_word, kErrBadIndex); tok = -1; }
    }

    st.m_ref = -INFINITY;
    st.shift = kRefShift;
    if (par == 1) {
        // the even-tile warpgroup takes the exact row maxima of key tile 0 and hands them over
        if (tile == 0) asm volatile("bar.sync 3, 256;" ::: "memory");
        else asm volatile("bar.sync 4, 256;" ::: "memory");
        st.m_ref = *st.ref_x;
    }
    for (int j = par; j < n_tiles; j += kSplit) softmax_step<C, kSpeculate>(st, j, j);
    wait_bar(st.bar_done, 0, abort_flag, p.err_word);            // every P V of this query tile has landed
    if constexpr (C::kOnes) {
        // the row sum came out of the tensor core with O; one that passed the limit (or is inf / NaN) means that
        // the reference was too low somewhere along the row
        tc_fence_after();
        uint32_t o[8];
        tmem_ld8(st.t_o + C::kOnesCol, o);
        tc_wait_ld();
        st.l_sum = __uint_as_float(o[0]);
        if (__any_sync(0xffffffffu, !(st.l_sum <= kTileSumLimit))) *redo_flag = 1;
    }
    pass_sync<C>();
    if (*redo_flag) {
        // a tile overflowed somewhere in the CTA: exact row maxima first, then the whole pass again
        st.m_ref = -INFINITY;
        for (int j = par; j < n_tiles; j += kSplit) softmax_step<C, kMaxOnly>(st, j, n_tiles + j);
        xchg[wtid + par * kBlockM].x = st.m_ref;
        if (tile == 0) asm volatile("bar.sync 1, 256;" ::: "memory");
        else asm volatile("bar.sync 2, 256;" ::: "memory");
        st.m_ref = fmaxf(xchg[wtid].x, xchg[wtid + kBlockM].x);
        st.shift = 0.f;
        st.l_sum = 0.f;
        for (int j = par; j < n_tiles; j += kSplit) softmax_step<C, kExact>(st, j, 2 * n_tiles + j);
        wait_bar(st.bar_done, 1, abort_flag, p.err_word);
        if constexpr (C::kOnes) {
            tc_fence_after();
            uint32_t o[8];
            tmem_ld8(st.t_o + C::kOnesCol, o);
            tc_wait_ld();
            st.l_sum = __uint_as_float(o[0]);
        }
    }

    // ------------------------------------------------ epilogue: normalise and scatter
    tc_fence_after();
    // both warpgroups accumulated into one O against one reference: add the row sums, split the columns
    float l_sum = st.l_sum;                                      // with the ones column: the row's whole sum already
    if constexpr (!C::kOnes) {
        xchg[wtid + par * kBlockM].y = st.l_sum;
        if (tile == 0) asm volatile("bar.sync 1, 256;" ::: "memory");
        else asm volatile("bar.sync 2, 256;" ::: "memory");
        l_sum = xchg[wtid].y + xchg[wtid + kBlockM].y;
    }
    constexpr int ncol = C::kMain / 2;                           // O columns this thread writes
    const int col0 = par * ncol;
    const float inv_l = 1.0f / l_sum;
    if (part >= 0) {
        // a share of the keys only: the normalised row and its LSE go to the workspace in fp32 (every row of the tile,
        // listed or not; the merge knows which ones count).  A CTA that gave up marks its rows with NaN.
        const size_t prow = (size_t)part * (C::kTilesM * kBlockM) + tile * kBlockM + wtid;
        float *po = p.part_o + prow * C::kDH;
        if (par == 0)
            p.part_lse[prow] = *abort_flag ? __int_as_float(0x7fc00000) : st.m_ref * p.scale + st.shift * 0.6931471805599453f + logf(l_sum);
#pragma unroll
        for (int cc = 0; cc < ncol; cc += 32) {
            const int c = col0 + cc;
            uint32_t o[32];
            tmem_ld32(st.t_o + c, o);
            tc_wait_ld();
#pragma unroll
            for (int v = 0; v < 8; ++v)
                *reinterpret_cast<float4 *>(po + c + v * 4) = make_float4(__uint_as_float(o[4 * v]) * inv_l, __uint_as_float(o[4 * v + 1]) * inv_l,
                                                                           __uint_as_float(o[4 * v + 2]) * inv_l, __uint_as_float(o[4 * v + 3]) * inv_l);
        }
        if (C::kTail && par == kSplit - 1) {
            uint32_t o[8];
            tmem_ld8(st.t_o + C::kMain, o);
            tc_wait_ld();
#pragma unroll
            for (int v = 0; v < 2; ++v)
                *reinterpret_cast<float4 *>(po + C::kMain + v * 4) = make_float4(__uint_as_float(o[4 * v]) * inv_l, __uint_as_float(o[4 * v + 1]) * inv_l,
                                                                                  __uint_as_float(o[4 * v + 2]) * inv_l, __uint_as_float(o[4 * v + 3]) * inv_l);
        }
        return;
    }
    __nv_bfloat16 *dst = nullptr;
    long long orow_ok = -1;                                      // this thread's output row, or -1: nothing is written
    if (tok >= 0 && !*abort_flag) {
        const size_t orow = p.compact ? ((size_t)b * p.M + m) : ((size_t)b * p.N_tok + tok);
        orow_ok = (long long)orow;
        dst = p.out + (orow * p.H + h) * C::kDH;
        if (p.lse_out && par == 0) {
            const size_t li = p.compact ? (((size_t)b * p.H + h) * p.M + m) : (((size_t)b * p.H + h) * p.N_tok + tok);
            p.lse_out[li] = st.m_ref * p.scale + st.shift * 0.6931471805599453f + logf(l_sum);
        }
    }
    // A thread owns a row: stored directly, a warp's 16-byte pieces would land in 32 different lines per instruction.
    // They go through shared memory instead and leave as 64 contiguous bytes per row, 8 rows per instruction: lane l
    // moves piece l & 3 of rows (l >> 2) + 8 j (pieces swizzled by the row: no bank conflicts either way).  The
    // staging area is this warp's 2 KB of its query tile's Q rows, which only this tile's MMAs read, and those are done.
    // (Not at head_dim 72: measured 3.5 % slower there with it, against +0.5-0.7 % at head_dim 64.)
    constexpr bool kStagedStores = C::kDH != 72;
    uint8_t *stage = sQ_gen + (par * 4 + warp) * 2048;
    static_assert(2 * 4 * 2048 <= C::kQTileBytes, "eight warps stage through their query tile's Q rows");
    const int lane = wtid & 31, q4 = lane & 3;
#pragma unroll
    for (int cc = 0; cc < ncol; cc += 32) {
        const int c = col0 + cc;
        uint32_t o[32];
        tmem_ld32(st.t_o + c, o);
        tc_wait_ld();
        if constexpr (!kStagedStores) {
            if (dst) {
#pragma unroll
                for (int v = 0; v < 4; ++v) {
                    uint32_t w[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        __nv_bfloat162 v2 = __floats2bfloat162_rn(__uint_as_float(o[v * 8 + 2 * i]) * inv_l, __uint_as_float(o[v * 8 + 2 * i + 1]) * inv_l);
                        w[i] = *reinterpret_cast<uint32_t *>(&v2);
                    }
                    *reinterpret_cast<uint4 *>(dst + c + v * 8) = make_uint4(w[0], w[1], w[2], w[3]);
                }
            }
        } else {
#pragma unroll
            for (int v = 0; v < 4; ++v) {
                uint32_t w[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    __nv_bfloat162 v2 = __floats2bfloat162_rn(__uint_as_float(o[v * 8 + 2 * i]) * inv_l, __uint_as_float(o[v * 8 + 2 * i + 1]) * inv_l);
                    w[i] = *reinterpret_cast<uint32_t *>(&v2);
                }
                *reinterpret_cast<uint4 *>(stage + lane * 64 + ((v ^ ((lane >> 1) & 3)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
            }
            __syncwarp();
#pragma unroll
            for (int jj = 0; jj < 4; ++jj) {
                const int r = (lane >> 2) + 8 * jj;
                const long long orow_r = __shfl_sync(0xffffffffu, orow_ok, r);
                const uint4 t = *reinterpret_cast<const uint4 *>(stage + r * 64 + ((q4 ^ ((r >> 1) & 3)) << 4));
                if (orow_r >= 0) *reinterpret_cast<uint4 *>(p.out + ((size_t)orow_r * p.H + h) * C::kDH + c + q4 * 8) = t;
            }
            __syncwarp();
        }
    }
    if (C::kTail && par == kSplit - 1) {
        uint32_t o[8], w[4];
        tmem_ld8(st.t_o + C::kMain, o);
        tc_wait_ld();
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            __nv_bfloat162 v2 = __floats2bfloat162_rn(__uint_as_float(o[2 * i]) * inv_l, __uint_as_float(o[2 * i + 1]) * inv_l);
            w[i] = *reinterpret_cast<uint32_t *>(&v2);
        }
        if (dst) *reinterpret_cast<uint4 *>(dst + C::kMain) = make_uint4(w[0], w[1], w[2], w[3]);
    }
}

template <class C>
__global__ void __launch_bounds__(C::kThreads, C::kCtasPerSM)
sparse_attn_kernel(const __grid_constant__ CUtensorMap tmap_k, const __grid_constant__ CUtensorMap tmap_v,
                   const __grid_constant__ CUtensorMap tmap_k_tail, const __grid_constant__ CUtensorMap tmap_v_tail, const Params p)
{
    constexpr int kTilesM = C::kTilesM;
    constexpr uint32_t kTmemCols = C::kTmemCols;
    constexpr int kSBufs = C::kSBufs, kAhead = C::kAhead;
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    __shared__ volatile int redo_flag;
    __shared__ float2 xchg[C::kTilesM][2 * kBlockM];

    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    const uint32_t sQ = smem_base;
    const uint32_t sK = sQ + kTilesM * C::kQTileBytes;
    const uint32_t sV = sK + C::kStagesK * C::kTileBytes;
    const uint32_t sOnes = sV + C::kStagesV * C::kTileBytes;       // [key tile x 16 columns] bf16, 32-byte swizzle, column 0 = 1
    const uint32_t bars = sOnes + C::kOnesBytes;
    Bars bar;
    bar.q = bars; bar.s = bars + 16; bar.p = bars + 80; bar.done = bars + 144;
    bar.kf = bars + 160;
    bar.ke = bar.kf + 8 * C::kStagesK;
    bar.vf = bar.ke + 8 * C::kStagesK;
    bar.ve = bar.vf + 8 * C::kStagesV;
    static_assert(160 + 16 * (C::kStagesK + C::kStagesV) <= C::kBarBytes, "barrier area too small");

    const int tid = threadIdx.x;
    const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);        // warp-uniform
    constexpr int kBlockN = C::kBlockN;
    int unit = blockIdx.x, kpart = 0, ksplit = 1;
    int part = -1;                                                 // >= 0: this CTA takes a share of the keys only
    if (unit >= p.n_full) {
        part = unit - p.n_full;
        kpart = part % p.split; ksplit = p.split;
        unit = p.n_full + part / p.split;
    }
    const int m0 = (unit % p.tiles_x) * (kTilesM * kBlockM), h = p.h0 + (unit / p.tiles_x) % p.heads, b = unit / (p.tiles_x * p.heads);
    const int n_tiles_all = (p.N + kBlockN - 1) / kBlockN;
    const int tile0 = n_tiles_all * kpart / ksplit;                // first key tile of this CTA (split <= 8: no overflow)
    const int n_tiles = n_tiles_all * (kpart + 1) / ksplit - tile0;
    const int key0 = tile0 * kBlockN;
    // the last CTA of a head may have rows in its first query tile only: the second tile's warps and MMAs are skipped
    const int q_tiles = (m0 + kBlockM < p.M) ? kTilesM : 1;

    if constexpr (C::kOnes) {
        // row r: 32 bytes; the 16-byte unit that holds column 0 is unit (r >> 2) & 1 under the 32-byte swizzle
        uint8_t *ones = smem_gen + (sOnes - smem_base);
        for (int i = tid; i < kBlockN * 2; i += C::kThreads) {
            const int r = i >> 1, unit = i & 1;
            const uint32_t first = (unit == ((r >> 2) & 1)) ? 0x3F80u : 0u;      // bf16 1.0 in column 0
            *reinterpret_cast<uint4 *>(ones + r * 32 + unit * 16) = make_uint4(first, 0u, 0u, 0u);
        }
        fence_proxy_async_smem();
    }
    if (tid == 0) {
        abort_flag = 0;
        redo_flag = 0;
        for (int t = 0; t < kTilesM; ++t) {
            mbar_init(bar.q + 8 * t, 128 * kSplit);
            mbar_init(bar.done + 8 * t, 1);
            for (int u = 0; u < 4; ++u) { mbar_init(bar.s + 32 * t + 8 * u, 1); mbar_init(bar.p + 32 * t + 8 * u, 128); }
        }
        fence_barrier_init();
    }
    constexpr int kProducerWarp = C::kSoftmaxWarps, kIssuerWarp = C::kSoftmaxWarps + 1;
    // The producer warp sets up the K/V stage barriers itself and sends for the first kAhead K tiles and the first V
    // tile at once: their flight then runs under the TMEM allocation, the CTA-wide barrier and the gather of the Q rows
    // (nobody else touches these barriers or the stages before that barrier).
    if (warp == kProducerWarp) {
        if (elect_one()) {
            // a K/V stage is free once the issuer of every active query tile has committed its MMAs on it
            for (int s = 0; s < C::kStagesK; ++s) { mbar_init(bar.kf + 8 * s, 1); mbar_init(bar.ke + 8 * s, q_tiles); }
            for (int s = 0; s < C::kStagesV; ++s) { mbar_init(bar.vf + 8 * s, 1); mbar_init(bar.ve + 8 * s, q_tiles); }
            fence_barrier_init();
            for (int j = 0; j < kAhead && j < n_tiles; ++j) {
                mbar_arrive_expect_tx(bar.kf + 8 * j, C::kLoadBytes);
#pragma unroll
                for (int ch = 0; ch < C::kChunks; ++ch)
                    tma_load_4d(sK + j * C::kTileBytes + ch * C::kChunkBytes, &tmap_k, bar.kf + 8 * j, ch * 64, key0 + j * kBlockN, h, b);
                if (C::kTail)
                    tma_load_4d(sK + j * C::kTileBytes + C::kChunks * C::kChunkBytes, &tmap_k_tail, bar.kf + 8 * j, C::kMain, key0 + j * kBlockN, h, b);
            }
            mbar_arrive_expect_tx(bar.vf, C::kLoadBytes);
#pragma unroll
            for (int ch = 0; ch < C::kChunks; ++ch)
                tma_load_4d(sV + ch * C::kChunkBytes, &tmap_v, bar.vf, ch * 64, key0, h, b);
            if (C::kTail)
                tma_load_4d(sV + C::kChunks * C::kChunkBytes, &tmap_v_tail, bar.vf, C::kMain, key0, h, b);
        }
        __syncwarp();
    }
    if (warp == kIssuerWarp) {
        tmem_alloc(smem_u32(&tmem_slot), kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_slot;

    if (warp < C::kSoftmaxWarps) {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(C::kRegsSoftmax));
        const int wg = warp >> 2;
        const int tile = wg / kSplit, par = wg % kSplit;
        if (tile < q_tiles)
            softmax_role<C>(p, bar, tile, par, smem_gen + tile * C::kQTileBytes, tmem, m0 + tile * kBlockM, h, b, n_tiles, key0, part,
                             &abort_flag, &redo_flag, xchg[tile]);
        else pass_sync<C>();
    } else if (warp == kProducerWarp) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(C::kRegsOther));
        // ------------------------------------------------ TMA producer (warp-uniform, one elected lane issues)
        if (elect_one()) {
            prefetch_tensormap(&tmap_k); prefetch_tensormap(&tmap_v);
            if (C::kTail) { prefetch_tensormap(&tmap_k_tail); prefetch_tensormap(&tmap_v_tail); }
        }
        // g: running count of K (or V) tiles over all passes: stage g % kStages, phase (g / kStages) & 1
        auto load_k = [&](int g, int j) {
            const int st = g % C::kStagesK;
            wait_bar(bar.ke + 8 * st, ((g / C::kStagesK) & 1) ^ 1, &abort_flag, p.err_word);
            if (elect_one()) {
                mbar_arrive_expect_tx(bar.kf + 8 * st, C::kLoadBytes);
#pragma unroll
                for (int ch = 0; ch < C::kChunks; ++ch)
                    tma_load_4d(sK + st * C::kTileBytes + ch * C::kChunkBytes, &tmap_k, bar.kf + 8 * st, ch * 64, key0 + j * kBlockN, h, b);
                if (C::kTail)
                    tma_load_4d(sK + st * C::kTileBytes + C::kChunks * C::kChunkBytes, &tmap_k_tail, bar.kf + 8 * st, C::kMain, key0 + j * kBlockN, h, b);
            }
            __syncwarp();
        };
        auto load_v = [&](int g, int j) {
            const int st = g % C::kStagesV;
            wait_bar(bar.ve + 8 * st, ((g / C::kStagesV) & 1) ^ 1, &abort_flag, p.err_word);
            if (elect_one()) {
                mbar_arrive_expect_tx(bar.vf + 8 * st, C::kLoadBytes);
#pragma unroll
                for (int ch = 0; ch < C::kChunks; ++ch)
                    tma_load_4d(sV + st * C::kTileBytes + ch * C::kChunkBytes, &tmap_v, bar.vf + 8 * st, ch * 64, key0 + j * kBlockN, h, b);
                if (C::kTail)
                    tma_load_4d(sV + st * C::kTileBytes + C::kChunks * C::kChunkBytes, &tmap_v_tail, bar.vf + 8 * st, C::kMain, key0 + j * kBlockN, h, b);
            }
            __syncwarp();
        };
        // K runs kAhead tiles ahead of V: K_{j+kAhead} is consumed next to V_j.  The max-only pass needs no V.
        auto produce_pass = [&](int pass) {
            const int gk0 = pass * n_tiles, gv0 = (pass == kExact) ? n_tiles : 0;
            const bool sent = pass == kSpeculate;        // the first K tiles and V tile of this pass are on their way already
            for (int j = 0; j < kAhead && j < n_tiles; ++j) if (!sent) load_k(gk0 + j, j);
            for (int j = 0; j < n_tiles; ++j) {
                if (j + kAhead < n_tiles) load_k(gk0 + j + kAhead, j + kAhead);
                if (pass != kMaxOnly && !(sent && j == 0)) load_v(gv0 + j, j);
            }
        };
        produce_pass(kSpeculate);
        int k_loads = n_tiles, v_loads = n_tiles;
        pass_sync<C>();
        if (redo_flag) {
            produce_pass(kMaxOnly);
            produce_pass(kExact);
            k_loads = 3 * n_tiles; v_loads = 2 * n_tiles;
        }
        // every copy issued above must have landed before the CTA's shared memory is released
        for (int g = (k_loads > C::kStagesK ? k_loads - C::kStagesK : 0); g < k_loads; ++g)
            wait_bar(bar.kf + 8 * (g % C::kStagesK), (g / C::kStagesK) & 1, &abort_flag, p.err_word);
        for (int g = (v_loads > C::kStagesV ? v_loads - C::kStagesV : 0); g < v_loads; ++g)
            wait_bar(bar.vf + 8 * (g % C::kStagesV), (g / C::kStagesV) & 1, &abort_flag, p.err_word);
    } else if (warp == kIssuerWarp || warp == kIssuerWarp + 1) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(C::kRegsOther));
        // ------------------------------------------------ MMA issuer (warp-uniform, one elected lane issues)
        constexpr uint32_t idesc_qk = idesc_bf16(kBlockM, kBlockN, false);
        constexpr uint32_t idesc_pv = idesc_bf16(kBlockM, C::kMain, true);
        constexpr uint32_t idesc_pv_tail = idesc_bf16(kBlockM, 16, true);
        // S[t][g % kSBufs] = Q_t K^T of the key tile in shared memory at kbase (one elected lane); g counts the
        // S-buffer uses of the query tile over all passes
        auto issue_qk = [&](int t, int g, uint32_t kbase) {
            const int u = g % kSBufs;
#pragma unroll
            for (int ks = 0; ks < C::kMain / 16; ++ks)
                mma_ss(tmem + (t * kSBufs + u) * kBlockN,
                       smem_desc(sQ + t * C::kQTileBytes + (ks >> 2) * C::kQChunkBytes + (ks & 3) * 32, 16, 1024, kSwizzle128B),
                       smem_desc(kbase + (ks >> 2) * C::kChunkBytes + (ks & 3) * 32, 16, 1024, kSwizzle128B),
                       idesc_qk, ks > 0);
            if (C::kTail)      // columns 64..79 (72..79 are zero): one more K step on the 32-byte-swizzled chunks
                mma_ss(tmem + (t * kSBufs + u) * kBlockN,
                       smem_desc(sQ + t * C::kQTileBytes + C::kChunks * C::kQChunkBytes, 16, 256, kSwizzle32B),
                       smem_desc(kbase + C::kChunks * C::kChunkBytes, 16, 256, kSwizzle32B), idesc_qk, 1u);
            tc_commit(bar.s + 32 * t + 8 * u);
        };
        // One issuer warp per query tile, on different SM sub-partitions: the tcgen05 instructions of a
        // sub-partition's issuer slow the exponentials of the softmax warps that live there, so the load is spread.
        // All MMAs that touch one S buffer / O accumulator come from one thread, in order.
        const int t = warp - kIssuerWarp;
        const uint32_t o_col = C::kColO + t * C::kOStride;
        auto issue_pass = [&](int pass) {
            const bool with_v = pass != kMaxOnly;
            const int gs0 = pass * n_tiles, gk0 = pass * n_tiles, gv0 = (pass == kExact) ? n_tiles : 0;
            // prologue: S of the first kAhead key tiles
            for (int j = 0; j < kAhead && j < n_tiles; ++j) {
                const int st = (gk0 + j) % C::kStagesK;
                wait_bar(bar.kf + 8 * st, ((gk0 + j) / C::kStagesK) & 1, &abort_flag, p.err_word);
                tc_fence_after();
                if (elect_one()) {
                    issue_qk(t, gs0 + j, sK + st * C::kTileBytes);
                    tc_commit(bar.ke + 8 * st);
                }
                __syncwarp();
            }
            for (int j = 0; j < n_tiles; ++j) {
                const int sv = (gv0 + j) % C::kStagesV;
                const uint32_t vbase = sV + sv * C::kTileBytes;
                const int u = (gs0 + j) % kSBufs;
                const bool more = j + kAhead < n_tiles;
                const int sk = (gk0 + j + kAhead) % C::kStagesK;
                if (more) wait_bar(bar.kf + 8 * sk, ((gk0 + j + kAhead) / C::kStagesK) & 1, &abort_flag, p.err_word);
                if (with_v) wait_bar(bar.vf + 8 * sv, ((gv0 + j) / C::kStagesV) & 1, &abort_flag, p.err_word);
                // P of key tile j is in TMEM (max-only pass: S of key tile j has been read)
                wait_bar(bar.p + 32 * t + 8 * u, ((gs0 + j) / kSBufs) & 1, &abort_flag, p.err_word);
                tc_fence_after();
                if (elect_one()) {
                    if (with_v) {
#pragma unroll
                        for (int ks = 0; ks < kBlockN / 16; ++ks) {
                            mma_ts(tmem + o_col, tmem + (t * kSBufs + u) * kBlockN + ks * 8,
                                   smem_desc(vbase + ks * 2048, C::kChunkBytes, 1024, kSwizzle128B),
                                   idesc_pv, (j > 0 || ks > 0) ? 1u : 0u);
                            if (C::kTail)  // O columns 64..79 from the 16-column chunk of V
                                mma_ts(tmem + o_col + C::kMain, tmem + (t * kSBufs + u) * kBlockN + ks * 8,
                                       smem_desc(vbase + C::kChunks * C::kChunkBytes + ks * 512, 256, 256, kSwizzle32B),
                                       idesc_pv_tail, (j > 0 || ks > 0) ? 1u : 0u);
                            if (C::kOnes)  // the row sums: P times the column of ones
                                mma_ts(tmem + o_col + C::kOnesCol, tmem + (t * kSBufs + u) * kBlockN + ks * 8,
                                       smem_desc(sOnes + ks * 512, 256, 256, kSwizzle32B),
                                       idesc_pv_tail, (j > 0 || ks > 0) ? 1u : 0u);
                        }
                        tc_commit(bar.ve + 8 * sv);
                        if (j == n_tiles - 1) tc_commit(bar.done + 8 * t);        // the pass is done for this query tile
                    }
                    // the S buffer just consumed as P is free again (in-order pipe): refill it with key tile j+2
                    if (more) {
                        issue_qk(t, gs0 + j + kAhead, sK + sk * C::kTileBytes);
                        tc_commit(bar.ke + 8 * sk);
                    }
                }
                __syncwarp();
            }
        };
        if (t < q_tiles) {
            wait_bar(bar.q + 8 * t, 0, &abort_flag, p.err_word);
            issue_pass(kSpeculate);
        }
        pass_sync<C>();
        if (redo_flag && t < q_tiles) {
            issue_pass(kMaxOnly);
            issue_pass(kExact);
        }
    } else {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(C::kRegsOther));
        pass_sync<C>();
    }

    tc_fence_before();
    __syncthreads();
    if (warp == kIssuerWarp) tmem_dealloc(tmem, kTmemCols);
}

// Combines the key shares of the split units: row = sum_i w_i row_i with w_i = exp(lse_i - LSE), LSE = log sum_i exp(lse_i)
// (each share is a complete softmax over its own keys).  One thread per (row, 8 columns); grid (head_dim / 8, units).
template <int DH, int ROWS>
__global__ void __launch_bounds__(ROWS) merge_parts_kernel(const Params p)
{
    constexpr int kChunksRow = DH / 8;
    const int unit = p.n_full + blockIdx.y;
    const int m0 = (unit % p.tiles_x) * ROWS, h = p.h0 + (unit / p.tiles_x) % p.heads, b = unit / (p.tiles_x * p.heads);
    const int idx = blockIdx.x * ROWS + threadIdx.x;
    const int r = idx / kChunksRow, c = idx - r * kChunksRow;
    const int m = m0 + r;
    if (m >= p.M) return;
    const int tok = p.q_idx ? __ldg(p.q_idx + (size_t)b * p.M + m) : m;
    if ((unsigned)tok >= (unsigned)p.N_tok || (p.q_idx && m > 0 && __ldg(p.q_idx + (size_t)b * p.M + m - 1) >= tok)) return;   // reported by the attention kernel
    const size_t part0 = (size_t)blockIdx.y * p.split;
    float lse[8], mx = -INFINITY;
    bool gave_up = false;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        lse[i] = -INFINITY;
        if (i < p.split) {
            lse[i] = __ldg(p.part_lse + (part0 + i) * ROWS + r);
            gave_up |= lse[i] != lse[i];
            mx = fmaxf(mx, lse[i]);
        }
    }
    if (gave_up) return;                                            // a share was not finished (a wait ran out): the row stays as it is
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f}, wsum = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        if (i < p.split) {
            const float w = __expf(lse[i] - mx);
            wsum += w;
            const float4 *src = reinterpret_cast<const float4 *>(p.part_o + ((part0 + i) * ROWS + r) * DH + c * 8);
            const float4 a = __ldg(src), d = __ldg(src + 1);
            acc[0] += w * a.x; acc[1] += w * a.y; acc[2] += w * a.z; acc[3] += w * a.w;
            acc[4] += w * d.x; acc[5] += w * d.y; acc[6] += w * d.z; acc[7] += w * d.w;
        }
    }
    const float inv = 1.0f / wsum;
    uint32_t w4[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        __nv_bfloat162 v2 = __floats2bfloat162_rn(acc[2 * i] * inv, acc[2 * i + 1] * inv);
        w4[i] = *reinterpret_cast<uint32_t *>(&v2);
    }
    const size_t orow = p.compact ? ((size_t)b * p.M + m) : ((size_t)b * p.N_tok + tok);
    *reinterpret_cast<uint4 *>(p.out + (orow * p.H + h) * DH + c * 8) = make_uint4(w4[0], w4[1], w4[2], w4[3]);
    if (p.lse_out && c == 0) {
        const size_t li = p.compact ? (((size_t)b * p.H + h) * p.M + m) : (((size_t)b * p.H + h) * p.N_tok + tok);
        p.lse_out[li] = mx + logf(wsum);
    }
}

// ------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() { return reinterpret_cast<EncodeTiledFn>(tensor_map_encoder()); }

// K or V as a 4-D tensor (d, N, H, B) with 128-byte-swizzled boxes of 64 columns x 128 tokens
int32_t make_kv_map(CUtensorMap *map, const void *base, int B, int H, int N, int d,
                    int64_t sb, int64_t sh, int64_t sn, bool tail, int tile_keys)
{
    EncodeTiledFn enc = get_encode_fn();
    if (!enc) return fail(ASTRAEA_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
    cuuint64_t dims[4] = {(cuuint64_t)d, (cuuint64_t)N, (cuuint64_t)H, (cuuint64_t)B};
    cuuint64_t strides[3] = {(cuuint64_t)sn * 2, (cuuint64_t)sh * 2, (cuuint64_t)sb * 2};
    // 64 columns x one key tile, 128-byte swizzle; or the 16-column tail chunk (32-byte swizzle; columns past d read as zero)
    cuuint32_t box[4] = {tail ? 16u : 64u, (cuuint32_t)tile_keys, 1, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(base), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, tail ? CU_TENSOR_MAP_SWIZZLE_32B : CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(ASTRAEA_ERR_INVALID_ARG, "tensor map rejected (CUresult %d): check K/V strides and alignment", (int)r);
    return ASTRAEA_OK;
}

// The last, partial round of CTAs of a launch: its `units` CTAs are replaced by `split` CTAs each, every one with a
// share of the key tiles, and merged afterwards (split 1: nothing is split).
struct SplitPlan { int units = 0, split = 1; };

constexpr int kMaxSplit = 8;                 // shares per unit
constexpr int kMaxSplitParts = 2 * 148;      // shares per launch (what the workspace holds)
constexpr int kMinSplitKeyTiles = 16;        // key tiles per share at least

template <int DH, int TM>
int32_t launch_dh(const AttnArgs &a, cudaStream_t stream, SplitPlan plan = SplitPlan())
{
    using C = Cfg<DH, TM>;
    CUtensorMap mk, mv, mkt, mvt;
    int32_t rc = make_kv_map(&mk, a.k, a.B, a.H, a.N, a.d, a.k_sb, a.k_sh, a.k_sn, false, C::kBlockN);
    if (rc != ASTRAEA_OK) return rc;
    rc = make_kv_map(&mv, a.v, a.B, a.H, a.N, a.d, a.v_sb, a.v_sh, a.v_sn, false, C::kBlockN);
    if (rc != ASTRAEA_OK) return rc;
    mkt = mk; mvt = mv;
    if (C::kTail) {
        rc = make_kv_map(&mkt, a.k, a.B, a.H, a.N, a.d, a.k_sb, a.k_sh, a.k_sn, true, C::kBlockN);
        if (rc != ASTRAEA_OK) return rc;
        rc = make_kv_map(&mvt, a.v, a.B, a.H, a.N, a.d, a.v_sb, a.v_sh, a.v_sn, true, C::kBlockN);
        if (rc != ASTRAEA_OK) return rc;
    }
    static PerDeviceOnce attrs;                   // one per kernel instantiation; the attributes are per device
    if (attrs.run([] {
            cudaError_t e = cudaFuncSetAttribute(sparse_attn_kernel<C>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes);
            if (e == cudaSuccess)
                e = cudaFuncSetAttribute(sparse_attn_kernel<C>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
            return e;
        }) != cudaSuccess)
        return check_launch("astraea_sparse_attn (shared memory attribute)");
    Params p;
    p.q = reinterpret_cast<const __nv_bfloat16 *>(a.q);
    p.q_sb = a.q_sb; p.q_sh = a.q_sh; p.q_sn = a.q_sn;
    p.q_idx = a.q_idx; p.M = a.M;
    p.out = reinterpret_cast<__nv_bfloat16 *>(a.out);
    p.lse_out = a.lse_out;
    p.N = a.N; p.H = a.H; p.N_tok = a.N_tok;
    p.scale = a.scale;
    p.scale_log2 = a.scale * 1.4426950408889634f;
    p.compact = (a.flags & ASTRAEA_ATTN_COMPACT_OUT) ? 1 : 0;
    p.err_word = a.err_word;
    p.h0 = a.head_begin;
    p.tiles_x = (a.M + TM * kBlockM - 1) / (TM * kBlockM);
    p.heads = a.head_count > 0 ? a.head_count : a.H;
    const long long units = (long long)p.tiles_x * p.heads * a.B;
    if (units + (long long)plan.units * (plan.split - 1) > 0x7fffffffll) return fail(ASTRAEA_ERR_INVALID_ARG, "astraea_sparse_attn: too many CTAs");
    const bool split = TM == 2 && plan.split > 1 && plan.units > 0;
    p.n_full = (int)units - (split ? plan.units : 0);
    p.split = split ? plan.split : 1;
    p.part_o = p.part_lse = nullptr;
    if (split) {
        // workspace behind the error word: the LSEs of all shares, then their rows
        const size_t parts = (size_t)plan.units * plan.split, rows = parts * (TM * kBlockM);
        p.part_lse = reinterpret_cast<float *>(static_cast<char *>(a.split_ws));
        p.part_o = p.part_lse + (rows + 63) / 64 * 64;
    }
    const unsigned grid = (unsigned)(p.n_full + (split ? plan.units * plan.split : 0));
    sparse_attn_kernel<C><<<grid, C::kThreads, C::kSmemBytes, stream>>>(mk, mv, mkt, mvt, p);
    if (split) {
        static_assert((TM * kBlockM * (DH / 8)) % (TM * kBlockM) == 0, "whole blocks per unit");
        merge_parts_kernel<DH, TM * kBlockM><<<dim3(DH / 8, plan.units), TM * kBlockM, 0, stream>>>(p);
    }
    return check_launch("astraea_sparse_attn");
}

}  // namespace

// 256 bytes for the error word; behind them room for the key shares of a split last round of CTAs (fp32 rows and
// LSEs), an upper bound over every M' <= M of the same problem
static size_t split_bytes(long long parts, int d) { return (size_t)parts * (2 * kBlockM) * ((size_t)d * 4 + 4) + 256; }
static int max_split_of(int N) { const int s = ((N + 63) / 64) / kMinSplitKeyTiles; return s > kMaxSplit ? kMaxSplit : s; }

size_t attn_workspace_bytes(int B, int H, int N, int M, int d)
{
    const int s_max = max_split_of(N);
    if (s_max < 2 || M <= 0) return 256;
    const long long units = (long long)B * H * ((M + 2 * kBlockM - 1) / (2 * kBlockM));
    const long long parts = units * s_max < kMaxSplitParts ? units * s_max : kMaxSplitParts;
    return 256 + split_bytes(parts, d);
}

// ---------------------------------------------------------------- gathered keys / values
// The "select Q and K" ablation of the paper restricts keys and values to listed tokens.  The listed K and V
// rows are gathered into compact [B, M_kv, H, d] buffers in the workspace, and the attention kernel runs on them.
namespace {
__global__ void __launch_bounds__(256)
gather_kv_kernel(uint4 *__restrict__ dst, const __nv_bfloat16 *__restrict__ src, int64_t sb, int64_t sh, int64_t sn,
                 const int32_t *__restrict__ idx, int B, int H, int N, int M_kv, int vec_per_row, int *err_word)
{
    const long long total = (long long)B * M_kv * H * vec_per_row;
    for (long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x; t < total; t += (long long)gridDim.x * blockDim.x) {
        const int v = (int)(t % vec_per_row);
        long long r = t / vec_per_row;
        const int h = (int)(r % H); r /= H;
        const int m = (int)(r % M_kv);
        const int b = (int)(r / M_kv);
        const int tok = __ldg(idx + (size_t)b * M_kv + m);
        uint4 val = make_uint4(0, 0, 0, 0);
        if ((unsigned)tok < (unsigned)N) val = __ldg(reinterpret_cast<const uint4 *>(src + b * sb + tok * sn + h * sh) + v);
        else if (v == 0 && h == 0) atomicExch(err_word, kErrBadIndex);
        dst[t] = val;
    }
}
}  // namespace

size_t attn_kv_workspace_bytes(int B, int H, int M_kv, int d) {
    const size_t one = ((size_t)B * M_kv * H * d * 2 + 255) / 256 * 256;
    return 256 + 2 * one;
}

int32_t launch_sparse_attn_kv(AttnArgs a, const int32_t *kv_idx, int M_kv, void *workspace, cudaStream_t stream)
{
    const size_t one = ((size_t)a.B * M_kv * a.H * a.d * 2 + 255) / 256 * 256;
    char *ws = reinterpret_cast<char *>(workspace);
    uint4 *kc = reinterpret_cast<uint4 *>(ws + 256), *vc = reinterpret_cast<uint4 *>(ws + 256 + one);
    const int vec = a.d / 8;
    const long long total = (long long)a.B * M_kv * a.H * vec;
    const long long cap = (long long)sm_count() * 16;
    const int grid = (int)((total + 255) / 256 < cap ? (total + 255) / 256 : cap);
    gather_kv_kernel<<<grid, 256, 0, stream>>>(kc, reinterpret_cast<const __nv_bfloat16 *>(a.k), a.k_sb, a.k_sh, a.k_sn,
                                               kv_idx, a.B, a.H, a.N, M_kv, vec, a.err_word);
    gather_kv_kernel<<<grid, 256, 0, stream>>>(vc, reinterpret_cast<const __nv_bfloat16 *>(a.v), a.v_sb, a.v_sh, a.v_sn,
                                               kv_idx, a.B, a.H, a.N, M_kv, vec, a.err_word);
    int32_t rc = check_launch("astraea_sparse_attn (gather of K/V)");
    if (rc != ASTRAEA_OK) return rc;
    a.k = kc; a.v = vc;
    a.k_sb = a.v_sb = (int64_t)M_kv * a.H * a.d;
    a.k_sh = a.v_sh = a.d;
    a.k_sn = a.v_sn = (int64_t)a.H * a.d;
    a.N = M_kv;                       // keys; a.N_tok stays the token count of q / out
    return launch_sparse_attn(a, stream);
}

// Scratch of astraea_sparse_attn_noalloc: lives in the library image, so every GPU that loads the
// library holds these bytes until the process exits.  In host code this name is only a handle of
// the symbol, never a device address: the address comes from cudaGetSymbolAddress, per device.
static __device__ __align__(256) unsigned char g_noalloc_scratch[ASTRAEA_NOALLOC_SCRATCH_BYTES];

int32_t noalloc_scratch_address(void **scratch_out)
{
    // one-time set-up per device (with that device current): resolve the symbol to its device address
    static void *scratch_of_device[kMaxDevices] = {};
    static std::mutex mu;
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess || dev < 0 || dev >= kMaxDevices)
        return fail(ASTRAEA_ERR_CUDA, "astraea_sparse_attn_noalloc: no usable current device (%s)", cudaGetErrorString(e));
    std::lock_guard<std::mutex> lock(mu);
    if (!scratch_of_device[dev]) {
        void *ptr = nullptr;
        e = cudaGetSymbolAddress(&ptr, g_noalloc_scratch);
        if (e != cudaSuccess || !ptr)
            return fail(ASTRAEA_ERR_CUDA, "astraea_sparse_attn_noalloc: cudaGetSymbolAddress failed: %s", cudaGetErrorString(e));
        scratch_of_device[dev] = ptr;
    }
    *scratch_out = scratch_of_device[dev];
    return ASTRAEA_OK;
}

// ---------------------------------------------------------------- self-test of the bounded wait
// One warp waits, with the given limit, on an mbarrier that is initialised and that nothing ever arrives at: the wait
// must give up, raise the error word and return, and the context must stay usable.  This is the give-up path that
// every tcgen05 kernel of the library takes when a copy or an MMA never completes, run where nothing else is at stake.
namespace {
__global__ void __launch_bounds__(32) wait_selftest_kernel(int *err_word, uint64_t limit_ns, int *gave_up)
{
    __shared__ __align__(8) uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        ptx::mbar_init(ptx::smem_u32(&bar), 1);
        ptx::fence_barrier_init();
    }
    __syncwarp();
    wait_bar(ptx::smem_u32(&bar), 0, &abort_flag, err_word, limit_ns);
    __syncwarp();
    if (threadIdx.x == 0 && gave_up) *gave_up = abort_flag;
}
}  // namespace

int32_t launch_wait_selftest(int *err_word, uint64_t limit_ns, int *gave_up, cudaStream_t stream)
{
    wait_selftest_kernel<<<1, 32, 0, stream>>>(err_word, limit_ns, gave_up);
    return check_launch("astraea_selftest_wait");
}

// Which launch finishes first.  Large CTAs (two query tiles, one per SM) are dispatched in launch order onto the SMs;
// the last one of every (head, batch) is cheaper when it holds one query tile only (0.68 of a full one, measured).
// Their last round is usually partial: its CTAs can each be replaced by `split` CTAs with a share of the keys (a share
// costs its part of the unit plus ~3 % for the query gather, the pipeline fill and the fp32 rows it writes), merged by
// a small kernel afterwards.  Small CTAs (one query tile, two per SM, head_dim 64 / 72) all cost the same: `slowdown`
// times a large one, because two share the SM (measured: 1.05 at head_dim 64, 1.17 at 72).  All of this matters for
// launches of a few rounds only.
namespace {
struct Schedule { bool small = false; SplitPlan plan; };

double finish_time(long long units, int pairs, bool light_last, int n_sm, int tail_units, int split)
{
    // greedy dispatch in launch order: every CTA goes to the SM that is free first (a binary min-heap of busy times)
    double heap[kMaxSMs] = {};
    double finish = 0.0;
    auto put = [&](double cost) {
        const double t = heap[0] + cost;
        finish = t > finish ? t : finish;
        int i = 0;
        for (;;) {                                               // replace the root and sift it down
            const int l = 2 * i + 1, r = l + 1;
            int m = l;
            if (l >= n_sm) break;
            if (r < n_sm && heap[r] < heap[l]) m = r;
            if (heap[m] >= t) break;
            heap[i] = heap[m];
            i = m;
        }
        heap[i] = t;
    };
    for (long long c = 0; c < units; ++c) {
        const double cost = (light_last && c % pairs == pairs - 1) ? 0.68 : 1.0;
        if (c < units - tail_units) put(cost);
        else for (int i = 0; i < split; ++i) put(cost / split + 0.03);
    }
    return finish;
}

Schedule choose_schedule(const AttnArgs &a, double slowdown /* 0: no small CTAs */)
{
    Schedule out;
    const long long hb = (long long)(a.head_count > 0 ? a.head_count : a.H) * a.B;
    const int pairs = (a.M + 2 * kBlockM - 1) / (2 * kBlockM), tiles = (a.M + kBlockM - 1) / kBlockM;
    const bool light_last = a.M - (pairs - 1) * 2 * kBlockM <= kBlockM;
    const int n_sm = sm_count();
    const long long units = hb * pairs;
    // a handful of key tiles (cross-attention over the text tokens): a CTA is mostly set-up (barriers, TMEM, the query
    // gather, the epilogue), which two small CTAs per SM overlap with each other's key loop (measured on 226 keys,
    // 9001 queries x 48 heads: 121 against 137 us)
    if (slowdown > 0.0 && (a.N + 63) / 64 <= 8 && tiles > 1) { out.small = true; return out; }
    if (units > 16 * n_sm) return out;                           // many rounds: the granularity does not matter
    // a denoising loop repeats a few shapes: remember the last answers
    struct Memo { long long hb = -1; int M = -1, N = -1, n_sm = 0; double slowdown = 0.0; size_t ws = 0; Schedule answer; };
    constexpr int kMemo = 16;
    thread_local Memo memo[kMemo];
    thread_local int memo_next = 0;
    const size_t ws_key = (a.flags & ASTRAEA_ATTN_WHOLE_KEYS) ? 0 : a.split_ws_bytes;
    for (const Memo &e : memo)
        if (e.hb == hb && e.M == a.M && e.N == a.N && e.n_sm == n_sm && e.slowdown == slowdown && e.ws == ws_key) return e.answer;
    double best = finish_time(units, pairs, light_last, n_sm, 0, 1);
    const double whole = best;
    const int tail = (int)(units % n_sm);
    if (a.split_ws && tail > 0 && !(a.flags & ASTRAEA_ATTN_WHOLE_KEYS)) {
        for (int s = 2; s <= max_split_of(a.N); ++s) {
            if ((long long)tail * s > kMaxSplitParts || split_bytes((long long)tail * s, a.d) > a.split_ws_bytes) break;
            const double t = finish_time(units, pairs, light_last, n_sm, tail, s);
            if (t < 0.98 * whole && t < best) { best = t; out.plan.units = tail; out.plan.split = s; }
        }
    }
    if (slowdown > 0.0) {
        const double small = slowdown * (double)((hb * tiles + 2 * n_sm - 1) / (2 * n_sm));
        if (small < 0.97 * best) { out.small = true; out.plan = SplitPlan(); }
    }
    Memo &e = memo[memo_next];
    memo_next = (memo_next + 1) % kMemo;
    e.hb = hb; e.M = a.M; e.N = a.N; e.n_sm = n_sm; e.slowdown = slowdown; e.ws = ws_key; e.answer = out;
    return out;
}
}  // namespace

void attn_plan(const AttnArgs &a, int *small_ctas, int *split_units, int *split)
{
    const bool force_small = (a.flags & ASTRAEA_ATTN_SMALL_CTAS) != 0 && a.d != 128;
    const Schedule sc = force_small ? Schedule() : choose_schedule(a, a.d == 64 ? 1.05 : a.d == 72 ? 1.17 : 0.0);
    *small_ctas = (force_small || sc.small) ? 1 : 0;
    *split_units = *small_ctas ? 0 : sc.plan.units;
    *split = *small_ctas ? 1 : sc.plan.split;
}

int32_t launch_sparse_attn(const AttnArgs &a, cudaStream_t stream)
{
    const bool force_small = (a.flags & ASTRAEA_ATTN_SMALL_CTAS) != 0;
    switch (a.d) {
    case 64: {
        const Schedule sc = force_small ? Schedule() : choose_schedule(a, 1.05);
        return (force_small || sc.small) ? launch_dh<64, 1>(a, stream) : launch_dh<64, 2>(a, stream, sc.plan);
    }
    case 72: {
        const Schedule sc = force_small ? Schedule() : choose_schedule(a, 1.17);
        return (force_small || sc.small) ? launch_dh<72, 1>(a, stream) : launch_dh<72, 2>(a, stream, sc.plan);
    }
    case 128: return launch_dh<128, 2>(a, stream, choose_schedule(a, 0.0).plan);
    default: return fail(ASTRAEA_ERR_UNSUPPORTED, "head_dim %d is not supported", a.d);
    }
}

}  // namespace astraea
