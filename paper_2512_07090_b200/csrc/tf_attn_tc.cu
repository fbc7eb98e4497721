// Step a5 on the 5th-generation tensor cores: bf16 causal (optionally windowed) attention for
// retained tokens only, head_dim 128.
//
// One CTA owns 256 consecutive entries of a sequence's retained list for one query head, as two
// 128-row Q tiles that share every K/V tile -- or, on grouped-query shapes, the same 128 entries for
// two query heads of one KV group (then both tiles need the same K/V tiles with the same masks).
// Warp roles:
//   warps 0-3 / 4-7  softmax group of Q tile 0 / 1 (thread r owns row r of its tile)
//   warp 8           issues every tcgen05.mma (one lane)
//   warp 9           TMA producer: K and V tiles of 128 keys into a 4-slot ring (one lane)
//   warps 10-11      idle; they complete the warpgroup whose registers go to the softmax groups
// The query rows are gathered (they are scattered in the sequence) into shared memory in the
// 128-byte-swizzled K-major operand layout.  Per K/V tile j and Q tile i:
//     S_i = Q_i K_j^T      A, B from shared memory (K-major)            -> TMEM, 128 columns
//     O_i += P_i V_j       A = P_i from TMEM (bf16, written over S_i),  B = V as it lies in
//                          memory (MN-major)                            -> TMEM, 128 columns
// issued in the order PV_0(j), QK_0(j+1), PV_1(j), QK_1(j+1): the tensor pipe works on one Q tile
// while the other tile's softmax group runs its exponentials.  The pipe executes in issue order,
// so S_i(j+1) is never produced before PV_i(j) has consumed P_i(j), and once a softmax group sees
// S_i(j) it may rescale O_i (PV_i(j-1) is complete).
// Softmax (fp32): row r applies ITS OWN causal / window limits (a tile of retained rows spans
// about 128/(1-ratio) positions), keeps a running reference maximum that is only moved (and O_i
// only rescaled) when the tile maximum exceeds it by more than 2^8, and writes P as bf16 pairs
// straight back into TMEM.  A Q tile skips K/V tiles none of its rows can see.  The epilogue
// normalises, converts to bf16 and scatters rows to their token positions; rows of pruned tokens
// between two retained tokens are zeroed by the thread that owns the later one (Section 3.2:
// a skipped token's attention output is zero).
//
// Every mbarrier wait is bounded by a cycle budget; on expiry the CTA records TF_ERR_TIMEOUT,
// stops waiting, lets copies in flight land, releases its TMEM and exits.
#include <algorithm>

#include "tf_ptx.cuh"

namespace tf {
namespace {

constexpr int kTileM = 128;           // rows per Q tile
constexpr int kQTiles = 2;            // Q tiles per CTA
constexpr int kTileN = 128;           // keys per K/V tile
constexpr int kHalfBytes = 128 * 128; // one [128 rows][128 B] swizzled block (64 bf16 per row)
constexpr int kTileBytes = 2 * kHalfBytes;
constexpr int kSoftmaxThreads = kQTiles * kTileM;
constexpr int kThreads = kSoftmaxThreads + 128;   // third warpgroup: MMA warp, TMA warp, two idle warps
constexpr int kMmaWarp = kSoftmaxThreads / 32, kTmaWarp = kMmaWarp + 1;
constexpr uint32_t kTmemCols = 512;   // S0 | S1 | O0 | O1, 128 fp32 columns each
constexpr float kRescaleThreshold = 8.f;         // log2 units

struct TcParams {
    const __nv_bfloat16* Q; __nv_bfloat16* O;
    Strides3 qs, os;
    int S, Hq, Hkv, window;
    float scale_log2;
    const int32_t* kept_idx; const int32_t* n_kept;
    DevStatus* status;
    int compact;          // 1: K / V hold the retained tokens only, entry c = token kept_idx[c] (TF_KV_RETAINED)
    int n_row_blocks;     // CTAs per (batch, query head)
    int bh_group;         // CTA order: (batch, head) pairs are taken in groups of this many; within a group all of the
                          // heaviest row block first.  1 = all row blocks of a head together, n_bh = heaviest first over all heads
    int first_pair;       // row block the first CTA of a head takes: the last one expected to hold retained rows
    long long wait_cycles;   // budget of one mbarrier wait
};

// Two ways of giving the two softmax groups of a CTA their work:
//   shared (kSplit = false): two consecutive 128-row Q tiles; every K/V tile is loaded once and used by both.
//   split  (kSplit = true):  ONE 128-row Q tile; the groups take alternate K/V tiles and their partial
//                            results (O, maximum, sum) are merged at the end.  Twice as many, half as
//                            long CTAs: used when the shared form would leave SMs idle or unbalanced.
template <bool kSplit> struct Cfg {
    static constexpr int kQBufs = kSplit ? 1 : 2;         // Q tiles in shared memory
    static constexpr int kStages = kSplit ? 6 : 4;        // ring slots, filled in the order K(j), V(j), K(j+1), V(j+1), ...
    static constexpr int kRows = kQBufs * kTileM;         // retained rows per CTA
    static constexpr int kStep = kSplit ? 2 : 1;          // K/V tile stride of one softmax group
    // shared-memory map (dynamic, base aligned to 1024 B)
    static constexpr int kOffQ = 0;
    static constexpr int kOffRing = kOffQ + kQBufs * kTileBytes;
    static constexpr int kOffBar = kOffRing + kStages * kTileBytes;
    static constexpr int kSmemBytes = kOffBar + 256 + 1024;   // barriers + alignment slack
};

// CTAs start in index order.  Row blocks of a head differ in length by the causal triangle, so the heaviest should
// go first, over as many heads as possible (the grid then ends with short CTAs from many heads, which fill the SMs
// evenly); but the CTAs that run at the same time should find K and V in L2, which the row blocks of one head do (they
// read nearly the same keys) and those of different heads do not.  So the (batch, head) pairs are taken in groups whose
// K and V fit the L2 budget, and inside a group the order is: heaviest row block of every head, next row block, ...
__device__ __forceinline__ void cta_work_item(const TcParams& p, int& rb, int& bh) {
    const int n_bh = (int)(gridDim.x / (unsigned)p.n_row_blocks);
    const int per_group = p.bh_group * p.n_row_blocks;
    const int g = (int)blockIdx.x / per_group, within = (int)blockIdx.x - g * per_group;
    const int g_size = min(p.bh_group, n_bh - g * p.bh_group);     // the last group may be smaller
    rb = within / g_size;
    bh = g * p.bh_group + within % g_size;
}

// bounded wait; after the first expiry in this CTA nobody waits any more
__device__ __forceinline__ void mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, long long budget_cycles,
                                          DevStatus* status, unsigned long long where) {
    mbar_wait_bounded(bar, parity, abort_flag, budget_cycles, status, where);
}

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// packed fp32x2 arithmetic (two lanes per instruction) and the 3-input maximum
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
    uint64_t d;
    asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "f"(lo), "f"(hi));
    return d;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    uint32_t d;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}

// instruction descriptors: M=128, N=128; the P V product takes V as it lies in memory (MN-major)
constexpr uint32_t kIdescQK = idesc_bf16(128, false, false);
constexpr uint32_t kIdescPV = idesc_bf16(128, false, true);

// byte offset of 16-byte chunk cc (0..15) of row r inside a two-block [128][64]+[128][64] operand
__device__ __forceinline__ uint32_t swz(int r, int cc) {
    return (uint32_t)((cc >> 3) * kHalfBytes + r * 128 + (((cc & 7) ^ (r & 7)) << 4));
}


// One thread's share (a row of 128 scores) of one K/V tile of 128 keys starting at key j0: S from TMEM, masking by the
// row's own visible range lo .. hi, running reference maximum, exponentials, P as bf16 pairs back into TMEM over the first
// 64 columns of S, running sum.  O (when it exists already) is rescaled when the reference maximum moves.
__device__ __forceinline__ void softmax_tile(uint32_t tm_s, uint32_t tm_o, int lo, int hi, int j0, float scale_log2,
                                             bool have_o, float& m_ref, float& l_run) {
    uint32_t sreg[128];
#pragma unroll
    for (int c = 0; c < 4; ++c) tmem_ld32(tm_s + c * 32, sreg + c * 32);
    tmem_wait_ld();
    const bool full = (j0 >= lo) && (j0 + kTileN - 1 <= hi);
    if (!full) {   // columns below c_lo or above c_hi are invisible to this row: -inf
        const int c_lo = lo - j0, c_hi = hi - j0;
        if (c_lo <= 0) {
#pragma unroll
            for (int c = 0; c < 128; ++c) if (c > c_hi) sreg[c] = 0xff800000u;
        } else if (c_hi >= kTileN - 1) {
#pragma unroll
            for (int c = 0; c < 128; ++c) if (c < c_lo) sreg[c] = 0xff800000u;
        } else {
#pragma unroll
            for (int c = 0; c < 128; ++c) if (c < c_lo || c > c_hi) sreg[c] = 0xff800000u;
        }
    }
    float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};   // four chains, not one of 128
#pragma unroll
    for (int c = 0; c < 128; c += 8) {
#pragma unroll
        for (int u = 0; u < 4; ++u)
            mx4[u] = max3(mx4[u], __uint_as_float(sreg[c + 2 * u]), __uint_as_float(sreg[c + 2 * u + 1]));
    }
    const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
    __syncwarp();   // rows take different masking branches; the TMEM accesses below are warp-wide
    // move the reference maximum only when the tile maximum exceeds it by 2^8 or more
    const float m_tile = mx * scale_log2;
    const bool move = m_tile > m_ref + kRescaleThreshold;   // also true on the first visible key (m_ref = -inf)
    const float m_new = move ? m_tile : m_ref;
    const float corr = move ? ex2(m_ref - m_new) : 1.f;
    if (have_o && __any_sync(0xffffffffu, move)) {
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            uint32_t o[32];
            tmem_ld32(tm_o + c * 32, o);
            tmem_wait_ld();
#pragma unroll
            for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * corr);
            tmem_st32(tm_o + c * 32, o);
        }
    }
    m_ref = m_new;
    const float m_safe = (m_ref == -INFINITY) ? 0.f : m_ref;
    const uint64_t sc2 = pack2(scale_log2, scale_log2), nm2 = pack2(-m_safe, -m_safe);
    uint64_t acc[4] = {0ull, 0ull, 0ull, 0ull};
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        uint32_t pk[32];
#pragma unroll
        for (int c = 0; c < 32; ++c) {
            float x0, x1;
            unpack2(fma2(pack2(__uint_as_float(sreg[h * 64 + 2 * c]), __uint_as_float(sreg[h * 64 + 2 * c + 1])), sc2, nm2), x0, x1);
            const float p0 = ex2(x0), p1 = ex2(x1);
            acc[c & 3] = add2(acc[c & 3], pack2(p0, p1));
            pk[c] = pack_bf16(p0, p1);
        }
        tmem_st32(tm_s + h * 32, pk);   // P_i over the first 64 columns of S_i
    }
    float a0, a1, a2, a3;
    unpack2(add2(acc[0], acc[1]), a0, a1);
    unpack2(add2(acc[2], acc[3]), a2, a3);
    const float psum = (a0 + a1) + (a2 + a3);
    l_run = fmaf(l_run, corr, psum);
}

// kHpt = query heads per Q tile: 0 = the forms above (one head per CTA); 1, 2 = the head forms of the shared form for
// grouped-query shapes: a Q tile holds the same 128 / kHpt retained rows of kHpt query heads of one KV group (row r of
// the tile is head r / (128 / kHpt), entry r % (128 / kHpt)), and the CTA's second tile the next kHpt heads of that group.
template <bool kSplit, int kHpt = 0>
__global__ void __launch_bounds__(kThreads, 1)
attention_tc_kernel(const TcParams p, const __grid_constant__ CUtensorMap mapK, const __grid_constant__ CUtensorMap mapV) {
    static_assert(!(kSplit && kHpt > 0), "the head forms are variants of the shared form");
    static_assert(kHpt == 0 || kHpt == 1 || kHpt == 2, "one, two or four query heads per CTA");
    using C = Cfg<kSplit>;
    constexpr bool kHeads = kHpt > 0;
    // retained-list entries one CTA covers; kOneSpan: both softmax groups work on the SAME entries (the split form:
    // alternate K/V tiles; the head forms: different query heads of one KV group, so that the groups' K/V tile ranges and
    // masks coincide and no tile is ever worked on by one group alone)
    constexpr bool kOneSpan = kSplit || kHeads;
    constexpr int kTileRows = kHeads ? kTileM / kHpt : kTileM;   // retained-list entries per Q tile
    constexpr int kRows = kOneSpan ? kTileRows : C::kRows;
    constexpr int kStages = C::kStages, kOffQ = C::kOffQ, kOffRing = C::kOffRing, kOffBar = C::kOffBar, kStep = C::kStep;
    extern __shared__ uint8_t smem_raw[];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const uint32_t sbase = smem_u32(smem);
    const uint32_t bar_q = sbase + kOffBar;              // Q tiles written
    const uint32_t bar_full = bar_q + 8;                 // [kStages] ring slot filled by TMA
    const uint32_t bar_empty = bar_full + 8 * kStages;   // [kStages] ring slot consumed by the MMAs
    const uint32_t bar_s = bar_empty + 8 * kStages;      // [2] S_i ready
    const uint32_t bar_p = bar_s + 16;                   // [2] P_i written (and O_i rescaled)
    const uint32_t bar_o = bar_p + 16;                   // all MMAs done
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + kOffBar + 160);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + kOffBar + 168);
    // Barriers and TMEM need nothing from global memory: they are set up before the wait for the previous kernel,
    // which (the selection, one CTA per sequence) lets this grid become resident while it still runs.  Every way
    // out of the kernel from here on gives the TMEM columns back.
    if (tid == 0) {
        mbar_init(bar_q, kSoftmaxThreads);
        for (int i = 0; i < kStages; ++i) { mbar_init(bar_full + 8 * i, 1); mbar_init(bar_empty + 8 * i, 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(bar_s + 8 * i, 1); mbar_init(bar_p + 8 * i, kTileM); }
        mbar_init(bar_o, 1);
        *abort_flag = 0;
        mbar_fence_init();
    }
    __syncwarp();
    if (warp == kMmaWarp) tmem_alloc(smem_u32(tmem_slot), kTmemCols);
    grid_dependency_wait();   // kept_idx / n_kept come from the kernel before this one
    int rb, bh;
    cta_work_item(p, rb, bh);
    // Row blocks are taken from the heaviest expected one (the last with retained rows, a host-side estimate) down to
    // block 0, then the blocks above the estimate, which are normally empty: CTAs with nothing to do start last
    // instead of delaying the first wave of real work.  Any estimate gives a one-to-one assignment.
    int pair = p.first_pair - rb;
    if (pair < 0) pair += p.n_row_blocks;
    constexpr int kHeadsPerCta = kHeads ? 2 * kHpt : 1;
    const int qh = (bh % (p.Hq / kHeadsPerCta)) * kHeadsPerCta, b = bh / (p.Hq / kHeadsPerCta);   // first (or only) head
    const int nk = p.n_kept[b];
    const int slot0 = pair * kRows;
    const int32_t* kept = p.kept_idx + (size_t)b * p.S;
    __nv_bfloat16* Ob = p.O + (long long)b * p.os.b + (long long)qh * p.os.h;
    const uint4 zero4 = make_uint4(0, 0, 0, 0);
    if (slot0 >= max(nk, 1) || nk == 0) {   // no retained row in this block (CTA-uniform)
        if (slot0 < max(nk, 1)) {           // nothing retained at all: the whole head is zero
            for (int hh = 0; hh < kHeadsPerCta; ++hh)
                for (int i = tid; i < p.S * 16; i += kThreads)
                    *reinterpret_cast<uint4*>(Ob + (long long)hh * p.os.h + (long long)(i >> 4) * p.os.t + (i & 15) * 8) = zero4;
        }
        tc_fence_before();
        __syncthreads();
        tc_fence_after();
        if (warp == kMmaWarp) tmem_dealloc(*tmem_slot, kTmemCols);
        return;
    }

    // The softmax threads read the retained indices of the Q rows they will gather (16 lanes per 256-byte row, the
    // 8 warps take 16 rows per round) and of their own row now, next to the loads the set-up below waits for anyway:
    // one global round trip less between the set-up and the first Q K^T.
    constexpr int kRounds = C::kRows / 16;   // 16 rows per round over the CTA's Q tiles
    int tq[kRounds];
    int t_row = -1;
    if (warp < kMmaWarp) {
#pragma unroll
        for (int it = 0; it < kRounds; ++it) {
            const int rr = it * 16 + warp * 2 + (lane >> 4);           // row of the CTA's Q buffer (tile rr / 128)
            const int s_q = slot0 + (kHeads ? (rr & (kTileRows - 1)) : rr);
            tq[it] = s_q < nk ? kept[s_q] : -1;
        }
        const int slot_pre = slot0 + (kOneSpan ? 0 : (warp >> 2) * kTileM) + (tid & (kTileRows - 1));
        if (slot_pre < nk) t_row = kept[slot_pre];
    }

    // ---- which K/V tiles each Q tile needs (CTA-uniform) -------------------------------------------
    // group i works on tiles jb[i], jb[i] + kStep, ... < je[i]
    int jb[kQTiles], je[kQTiles];
#pragma unroll
    for (int i = 0; i < kQTiles; ++i) {
        const int s_lo = slot0 + (kOneSpan ? 0 : i * kTileM);
        if (s_lo < nk) {
            const int s_last = min(s_lo + kTileRows, nk) - 1;
            const int t_first = kept[s_lo], t_last = kept[s_last];
            int k_first = p.window > 0 ? max(0, t_first - p.window + 1) : 0;   // first key the tile's first row sees
            int k_last = t_last;                                                // last key its last row sees
            if (p.compact) {   // keys are entries of the retained list
                k_first = p.window > 0 ? first_kept_at_or_after(kept, s_lo + 1, k_first) : 0;
                k_last = s_last;
            }
            jb[i] = k_first / kTileN + (kSplit ? i : 0);
            je[i] = k_last / kTileN + 1;
        } else {
            jb[i] = je[i] = 0;
        }
    }
    const int n_q = kSplit ? 1 : ((je[1] > jb[1]) ? 2 : 1);   // Q tiles to gather
    const int J0 = jb[0], J1 = max(je[0], je[1]);   // rows ascend, so tile 0 starts first
    const int kh = qh / (p.Hq / p.Hkv);

    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    // registers move from the third warpgroup (which needs few) to the two softmax groups
    // (each setmaxnreg sits at the top of the branch it governs, so no later code sees both)
    if (warp >= kMmaWarp) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 72;");
    if (warp > kTmaWarp) {
        // ================================ zero fill (the two spare warps) ================================
        // rows of pruned tokens that precede a retained row of this CTA (and follow the last retained
        // one) are zero; 16 lanes write one row
        const int g4 = (tid - (kTmaWarp + 1) * 32) >> 4, l16 = tid & 15;
        const int s_end = min(slot0 + kRows, nk);
        for (int s_z = slot0 + g4; s_z < s_end; s_z += 4) {
            const int prev = s_z == 0 ? -1 : kept[s_z - 1], cur = kept[s_z];
            for (int hh = 0; hh < kHeadsPerCta; ++hh) {
                __nv_bfloat16* Oz = Ob + (long long)hh * p.os.h + l16 * 8;
                for (int t = prev + 1; t < cur; ++t) *reinterpret_cast<uint4*>(Oz + (long long)t * p.os.t) = zero4;
                if (s_z == nk - 1)
                    for (int t = cur + 1; t < p.S; ++t) *reinterpret_cast<uint4*>(Oz + (long long)t * p.os.t) = zero4;
            }
        }
    } else if (warp == kTmaWarp) {
        // ================================ TMA producer ================================================
        if (lane == 0) {
            int q = 0;
            for (int j = J0; j < J1; ++j) {
                for (int kv = 0; kv < 2; ++kv, ++q) {
                    const int st = q % kStages;
                    // the first K and V tiles go out at once; the rest of the ring is filled once the Q rows are in shared
                    // memory (nothing can consume it earlier, and a ring's worth of arriving tiles keeps the gather's
                    // shared-memory stores waiting)
                    if (q == 2) mbar_wait(bar_q, 0, abort_flag, p.wait_cycles, p.status, 11);
                    if (q >= kStages) mbar_wait(bar_empty + 8 * st, ((q / kStages) - 1) & 1, abort_flag, p.wait_cycles, p.status, 10);
                    const uint32_t dst = sbase + kOffRing + st * kTileBytes;
                    const CUtensorMap* map = kv ? &mapV : &mapK;
                    mbar_expect_tx(bar_full + 8 * st, kTileBytes);
                    tma_load_4d(dst, map, bar_full + 8 * st, 0, kh, j * kTileN, b);
                    tma_load_4d(dst + kHalfBytes, map, bar_full + 8 * st, 64, kh, j * kTileN, b);
                }
            }
        }
    } else if (warp == kMmaWarp) {
        // ================================ MMA issuer ==================================================
        if (lane == 0) {
            auto slot_of = [&](int j, int kv) { return (2 * (j - J0) + kv) % kStages; };
            auto par_of = [&](int j, int kv) { return ((2 * (j - J0) + kv) / kStages) & 1; };
            auto active = [&](int i, int j) { return j >= jb[i] && j < je[i]; };
            auto issue_qk = [&](int i, int j) {   // S_i = Q_i K_j^T : 8 steps of 16 dims
                const uint32_t kaddr = sbase + kOffRing + slot_of(j, 0) * kTileBytes;
                const uint32_t qaddr = sbase + kOffQ + (kSplit ? 0 : i) * kTileBytes;   // split: both groups share the Q tile
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) {
                    const uint32_t off = (kk >> 2) * kHalfBytes + (kk & 3) * 32;
                    mma_ss(tmem + i * 128, desc_kmajor(qaddr + off), desc_kmajor(kaddr + off), kIdescQK, kk > 0);
                }
                mma_commit(bar_s + 8 * i);
            };
            auto issue_pv = [&](int i, int j, bool first) {   // O_i (+)= P_i V_j : 8 steps of 16 keys
                const uint32_t vaddr = sbase + kOffRing + slot_of(j, 1) * kTileBytes;
#pragma unroll
                for (int kk = 0; kk < 8; ++kk)
                    mma_ts(tmem + 256 + i * 128, tmem + i * 128 + kk * 8, desc_mnmajor(vaddr + kk * 16 * 128, kHalfBytes), kIdescPV,
                           (!first || kk > 0) ? 1u : 0u);
            };
            mbar_wait(bar_q, 0, abort_flag, p.wait_cycles, p.status, 20);
            int done[kQTiles] = {0, 0};
            if constexpr (kSplit) {
                // tile j belongs to group (j - J0) & 1; order: QK_0(J0), QK_1(J0+1), then per tile PV(j), QK(j+2)
                for (int j = J0; j < min(J0 + 2, J1); ++j) {
                    mbar_wait(bar_full + 8 * slot_of(j, 0), par_of(j, 0), abort_flag, p.wait_cycles, p.status, 21);
                    tc_fence_after();
                    issue_qk(j - J0, j);
                    mma_commit(bar_empty + 8 * slot_of(j, 0));
                }
                for (int j = J0; j < J1; ++j) {
                    const int i = (j - J0) & 1;
                    mbar_wait(bar_full + 8 * slot_of(j, 1), par_of(j, 1), abort_flag, p.wait_cycles, p.status, 22);
                    mbar_wait(bar_p + 8 * i, done[i] & 1, abort_flag, p.wait_cycles, p.status, 24 + i);
                    tc_fence_after();
                    issue_pv(i, j, done[i] == 0);
                    ++done[i];
                    mma_commit(bar_empty + 8 * slot_of(j, 1));
                    if (j + 2 < J1) {
                        mbar_wait(bar_full + 8 * slot_of(j + 2, 0), par_of(j + 2, 0), abort_flag, p.wait_cycles, p.status, 23);
                        issue_qk(i, j + 2);
                        mma_commit(bar_empty + 8 * slot_of(j + 2, 0));
                    }
                }
            } else {
            mbar_wait(bar_full + 8 * slot_of(J0, 0), par_of(J0, 0), abort_flag, p.wait_cycles, p.status, 21);
            tc_fence_after();
            for (int i = 0; i < kQTiles; ++i)
                if (active(i, J0)) issue_qk(i, J0);
            mma_commit(bar_empty + 8 * slot_of(J0, 0));
            for (int j = J0; j < J1; ++j) {
                mbar_wait(bar_full + 8 * slot_of(j, 1), par_of(j, 1), abort_flag, p.wait_cycles, p.status, 22);
                if (j + 1 < J1) mbar_wait(bar_full + 8 * slot_of(j + 1, 0), par_of(j + 1, 0), abort_flag, p.wait_cycles, p.status, 23);
#pragma unroll
                for (int i = 0; i < kQTiles; ++i) {
                    if (active(i, j)) {
                        mbar_wait(bar_p + 8 * i, done[i] & 1, abort_flag, p.wait_cycles, p.status, 24 + i);
                        tc_fence_after();
                        issue_pv(i, j, done[i] == 0);
                        ++done[i];
                    }
                    if (i == kQTiles - 1) mma_commit(bar_empty + 8 * slot_of(j, 1));
                    if (j + 1 < J1 && active(i, j + 1)) issue_qk(i, j + 1);
                }
                if (j + 1 < J1) mma_commit(bar_empty + 8 * slot_of(j + 1, 0));
            }
            }
            mma_commit(bar_o);
        }
    }
    } else {
        // ================================ softmax groups ===============================================
        asm volatile("setmaxnreg.inc.sync.aligned.u32 216;");
        const int i = warp >> 2;                 // group: its Q tile (shared) or its half of the K/V tiles (split)
        const int r = tid & (kTileM - 1);        // row within the tile
        const int slot = slot0 + (kOneSpan ? 0 : i * kTileM) + (r & (kTileRows - 1));
        const bool valid = slot < nk;               // t_row (fetched above) is the row's token position, -1 if none
        int hi = t_row;                                                           // visible keys: lo .. hi
        int lo = (valid && p.window > 0) ? max(0, t_row - p.window + 1) : 0;
        if (p.compact && valid) {
            lo = p.window > 0 ? first_kept_at_or_after(kept, slot + 1, lo) : 0;
            hi = slot;
        }
        {
            // gather the CTA's Q rows into the swizzled K-major operand layout
            const int sub = lane >> 4, cc = lane & 15, w8 = tid >> 5;
            uint4 qv[kRounds];
            const __nv_bfloat16* qbase = p.Q + (long long)b * p.qs.b + (long long)qh * p.qs.h + cc * 8;
#pragma unroll
            for (int it = 0; it < kRounds; ++it) {   // head forms: rounds 8..15 fill the second tile, a round lies within one head
                const int hh = kHeads ? (it >> 3) * kHpt + ((it & 7) * 16) / kTileRows : 0;
                qv[it] = tq[it] >= 0 ? ldg16(qbase + (long long)hh * p.qs.h + (long long)tq[it] * p.qs.t) : zero4;
            }
#pragma unroll
            for (int it = 0; it < kRounds; ++it) {
                const int rr = it * 16 + w8 * 2 + sub;
                *reinterpret_cast<uint4*>(smem + kOffQ + (rr >> 7) * kTileBytes + swz(rr & (kTileM - 1), cc)) = qv[it];
            }
            fence_proxy_async();
            mbar_arrive(bar_q);
        }
        __syncwarp();
        const uint32_t tm_s = tmem + ((uint32_t)((warp & 3) * 32) << 16) + i * 128;   // this warp's lanes, S_i / P_i
        const uint32_t tm_o = tm_s + 256;                                               // O_i
        float m_ref = -INFINITY, l_run = 0.f;
        for (int j = jb[i]; j < je[i]; j += kStep) {
            const int c_it = (j - jb[i]) / kStep;
            const int j0 = j * kTileN;
            mbar_wait(bar_s + 8 * i, c_it & 1, abort_flag, p.wait_cycles, p.status, 30 + i);
            __syncwarp();
            tc_fence_after();
            softmax_tile(tm_s, tm_o, lo, hi, j0, p.scale_log2, c_it > 0, m_ref, l_run);
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(bar_p + 8 * i);
        }
        // ---- epilogue: O / l -> bf16 -> the row's token position --------------------------------------
        // A thread owns a row, and rows of retained tokens lie far apart in O: storing from the registers would
        // touch 32 different lines per warp instruction.  The rows are therefore staged in the shared memory of the
        // Q tile (nobody reads it once every MMA has completed; 16-byte chunks XOR-swizzled by the row) and written
        // out with 16 lanes per 256-byte row.  (maximum, sum) of the split form and the rows' token positions
        // travel through the first K/V ring slot, equally idle by now.
        if constexpr (kSplit) {
            // merge the two groups' partial results: both accumulators sit in the TMEM lanes of this row,
            // so each group finishes 64 of the 128 output columns
            mbar_wait(bar_o, 0, abort_flag, p.wait_cycles, p.status, 40);
            __syncwarp();
            tc_fence_after();
            float2* ml = reinterpret_cast<float2*>(smem + kOffRing);
            int* trow_s = reinterpret_cast<int*>(smem + kOffRing + 4096);
            ml[i * kTileM + r] = make_float2(m_ref, l_run);
            if (i == 0) trow_s[r] = t_row;                        // -1: no such row
            asm volatile("bar.sync 1, %0;" :: "n"(kSoftmaxThreads) : "memory");
            const float2 other = ml[(i ^ 1) * kTileM + r];
            const bool both = je[1] > jb[1];                       // group 1 had tiles (CTA-uniform)
            const float m0 = i == 0 ? m_ref : other.x, l0 = i == 0 ? l_run : other.y;   // group 0 always has a tile
            const float m1 = i == 0 ? other.x : m_ref, l1 = i == 0 ? other.y : l_run;
            const float m_all = both ? fmaxf(m0, m1) : m0;
            const float e0 = ex2(m0 - m_all), e1 = both ? ex2(m1 - m_all) : 0.f;
            const float inv = 1.f / (l0 * e0 + l1 * e1);
            const float w0 = e0 * inv, w1 = e1 * inv;
            const uint32_t tm_row = tmem + ((uint32_t)((warp & 3) * 32) << 16);
            uint8_t* stage = smem + kOffQ + r * 256;
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                uint32_t o0[32], o1[32];
                tmem_ld32(tm_row + 256 + i * 64 + c * 32, o0);
                if (both) tmem_ld32(tm_row + 384 + i * 64 + c * 32, o1);
                tmem_wait_ld();
#pragma unroll
                for (int v = 0; v < 4; ++v) {
                    float f[8];
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        f[e] = __uint_as_float(o0[8 * v + e]) * w0;
                        if (both) f[e] = fmaf(__uint_as_float(o1[8 * v + e]), w1, f[e]);
                    }
                    uint4 w;
                    w.x = pack_bf16(f[0], f[1]); w.y = pack_bf16(f[2], f[3]);
                    w.z = pack_bf16(f[4], f[5]); w.w = pack_bf16(f[6], f[7]);
                    *reinterpret_cast<uint4*>(stage + (((i * 8 + c * 4 + v) ^ (r & 15)) << 4)) = w;
                }
            }
            asm volatile("bar.sync 1, %0;" :: "n"(kSoftmaxThreads) : "memory");
            const int sub = tid >> 4, l16 = tid & 15;              // 256 threads: 16 rows per pass
#pragma unroll
            for (int pass = 0; pass < kTileM / 16; ++pass) {
                const int R = pass * 16 + sub, t_out = trow_s[R];
                if (t_out >= 0)
                    *reinterpret_cast<uint4*>(Ob + (long long)t_out * p.os.t + l16 * 8) =
                        *reinterpret_cast<const uint4*>(smem + kOffQ + R * 256 + ((l16 ^ (R & 15)) << 4));
            }
        } else if (i < n_q) {
            mbar_wait(bar_o, 0, abort_flag, p.wait_cycles, p.status, 40);
            __syncwarp();
            tc_fence_after();
            const float inv = 1.f / l_run;
            __nv_bfloat16* Oi = Ob + (kHeads ? (long long)(i * kHpt) * p.os.h : 0ll);   // this group's first head
            int* trow_s = reinterpret_cast<int*>(smem + kOffRing + 4096) + i * kTileM;
            trow_s[r] = t_row;
            uint8_t* stage = smem + kOffQ + i * kTileBytes + r * 256;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t o[32];
                tmem_ld32(tm_o + c * 32, o);
                tmem_wait_ld();
#pragma unroll
                for (int v = 0; v < 4; ++v) {
                    uint4 w;
                    w.x = pack_bf16(__uint_as_float(o[8 * v + 0]) * inv, __uint_as_float(o[8 * v + 1]) * inv);
                    w.y = pack_bf16(__uint_as_float(o[8 * v + 2]) * inv, __uint_as_float(o[8 * v + 3]) * inv);
                    w.z = pack_bf16(__uint_as_float(o[8 * v + 4]) * inv, __uint_as_float(o[8 * v + 5]) * inv);
                    w.w = pack_bf16(__uint_as_float(o[8 * v + 6]) * inv, __uint_as_float(o[8 * v + 7]) * inv);
                    *reinterpret_cast<uint4*>(stage + (((c * 4 + v) ^ (r & 15)) << 4)) = w;
                }
            }
            asm volatile("bar.sync %0, %1;" :: "r"(2 + i), "n"(kTileM) : "memory");   // this group's 128 threads
            const int sub = r >> 4, l16 = r & 15;                  // 128 threads: 8 rows per pass
#pragma unroll
            for (int pass = 0; pass < kTileM / 8; ++pass) {
                const int R = pass * 8 + sub, t_out = trow_s[R];
                if (t_out >= 0)
                    *reinterpret_cast<uint4*>(Oi + (long long)(R / kTileRows) * p.os.h + (long long)t_out * p.os.t + l16 * 8) =
                        *reinterpret_cast<const uint4*>(smem + kOffQ + i * kTileBytes + R * 256 + ((l16 ^ (R & 15)) << 4));
            }
        }
    }
    __syncwarp();
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {   // a wait gave up: give copies and MMAs still in flight time to land before leaving
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000ll) { }
        __syncthreads();
    }
    if (warp == kMmaWarp) tmem_dealloc(tmem, kTmemCols);
}

// ---------------------------------------------------------------------------------------------------------
// Single form: ONE 128-row Q tile and ONE softmax group per CTA -- 256 threads, 256 TMEM columns (S | O) and 96 KiB
// of shared memory (the Q tile, one K slot, one V slot), so that TWO CTAs share an SM.  What the two softmax groups
// of the other forms do for each other inside a CTA (one exponentiates while the tensor pipe works for the other),
// two independent CTAs do here, and in addition the set-up, Q gather and epilogue of one CTA run under the steady
// state of its neighbour: the fixed cost per CTA, a third of all SM time on small problems, is no longer idle time.
// Every Q tile streams its own K/V tiles (as in the split form), so this form suits problems whose K/V traffic the
// L2 can feed twice over.  Warp roles: warps 0-3 softmax (thread r owns row r), warp 4 issues the products, warp 5
// the TMA loads, warps 6-7 zero the output rows of pruned tokens.
//   K(j+1) is requested as soon as Q K_j^T has read K(j), V(j+1) as soon as P V_j has read V(j): with one slot each
//   the loads run under the softmax of tile j and the products of the neighbouring CTA.
// ---------------------------------------------------------------------------------------------------------
constexpr int kThreads1 = 256;
constexpr int kMmaWarp1 = 4, kTmaWarp1 = 5;
constexpr uint32_t kTmemCols1 = 256;
constexpr int kOffQ1 = 0, kOffK1 = kTileBytes, kOffV1 = 2 * kTileBytes, kOffBar1 = 3 * kTileBytes;
constexpr int kSmemBytes1 = kOffBar1 + 256;      // the dynamic segment must start 1024-byte aligned (checked)
constexpr int kRegs1 = 128;                      // registers per thread at launch: 256 x 128 = 128 x 200 + 128 x 56

__global__ void __launch_bounds__(kThreads1, 2)
attention_tc_single_kernel(const TcParams p, const __grid_constant__ CUtensorMap mapK, const __grid_constant__ CUtensorMap mapV) {
    extern __shared__ uint8_t smem[];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t sbase = smem_u32(smem);
    if (sbase & 1023u) {   // the swizzled operand layout needs it; nothing has been started yet
        if (tid == 0) report_error(p.status, TF_ERR_TIMEOUT, 399);
        return;
    }
    const uint32_t bar_q = sbase + kOffBar1;              // Q tile written
    const uint32_t bar_fk = bar_q + 8, bar_fv = bar_q + 16;   // K / V slot filled by TMA
    const uint32_t bar_ek = bar_q + 24, bar_ev = bar_q + 32;  // K / V slot consumed by the products
    const uint32_t bar_s = bar_q + 40, bar_p = bar_q + 48, bar_o = bar_q + 56;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + kOffBar1 + 64);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + kOffBar1 + 72);
    if (tid == 0) {
        mbar_init(bar_q, kTileM);
        mbar_init(bar_fk, 1); mbar_init(bar_fv, 1); mbar_init(bar_ek, 1); mbar_init(bar_ev, 1);
        mbar_init(bar_s, 1); mbar_init(bar_p, kTileM); mbar_init(bar_o, 1);
        *abort_flag = 0;
        mbar_fence_init();
    }
    __syncwarp();
    if (warp == kMmaWarp1) tmem_alloc(smem_u32(tmem_slot), kTmemCols1);
    grid_dependency_wait();   // kept_idx / n_kept come from the kernel before this one
    int rb, bh;
    cta_work_item(p, rb, bh);
    int blk = p.first_pair - rb;          // heaviest expected row block first, blocks expected to be empty last
    if (blk < 0) blk += p.n_row_blocks;
    const int qh = bh % p.Hq, b = bh / p.Hq;
    const int nk = p.n_kept[b];
    const int slot0 = blk * kTileM;
    const int32_t* kept = p.kept_idx + (size_t)b * p.S;
    __nv_bfloat16* Ob = p.O + (long long)b * p.os.b + (long long)qh * p.os.h;
    const uint4 zero4 = make_uint4(0, 0, 0, 0);
    if (slot0 >= max(nk, 1) || nk == 0) {   // no retained row in this block (CTA-uniform)
        if (slot0 < max(nk, 1)) {           // nothing retained at all: the whole head is zero
            for (int i = tid; i < p.S * 16; i += kThreads1)
                *reinterpret_cast<uint4*>(Ob + (long long)(i >> 4) * p.os.t + (i & 15) * 8) = zero4;
        }
        tc_fence_before();
        __syncthreads();
        tc_fence_after();
        if (warp == kMmaWarp1) tmem_dealloc(*tmem_slot, kTmemCols1);
        return;
    }
    // retained indices of the Q rows this thread gathers (16 lanes per 256-byte row, the 4 softmax warps take 8 rows per
    // round) and of its own row
    constexpr int kRounds = kTileM / 8;
    int tq[kRounds];
    int t_row = -1;
    if (warp < kMmaWarp1) {
#pragma unroll
        for (int it = 0; it < kRounds; ++it) {
            const int s_q = slot0 + it * 8 + warp * 2 + (lane >> 4);
            tq[it] = s_q < nk ? kept[s_q] : -1;
        }
        if (slot0 + tid < nk) t_row = kept[slot0 + tid];
    }
    // which K/V tiles the Q tile needs (CTA-uniform): J0 .. J1 - 1
    int J0, J1;
    {
        const int s_last = min(slot0 + kTileM, nk) - 1;
        const int t_first = kept[slot0], t_last = kept[s_last];
        int k_first = p.window > 0 ? max(0, t_first - p.window + 1) : 0;
        int k_last = t_last;
        if (p.compact) {   // keys are entries of the retained list
            k_first = p.window > 0 ? first_kept_at_or_after(kept, slot0 + 1, k_first) : 0;
            k_last = s_last;
        }
        J0 = k_first / kTileN;
        J1 = k_last / kTileN + 1;
    }
    const int kh = qh / (p.Hq / p.Hkv);

    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp >= kMmaWarp1) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 56;");
        if (warp > kTmaWarp1) {
            // ================================ zero fill ====================================================
            const int g4 = (tid - (kTmaWarp1 + 1) * 32) >> 4, l16 = tid & 15;
            const int s_end = min(slot0 + kTileM, nk);
            for (int s_z = slot0 + g4; s_z < s_end; s_z += 4) {
                const int prev = s_z == 0 ? -1 : kept[s_z - 1], cur = kept[s_z];
                for (int t = prev + 1; t < cur; ++t) *reinterpret_cast<uint4*>(Ob + (long long)t * p.os.t + l16 * 8) = zero4;
                if (s_z == nk - 1)
                    for (int t = cur + 1; t < p.S; ++t) *reinterpret_cast<uint4*>(Ob + (long long)t * p.os.t + l16 * 8) = zero4;
            }
        } else if (warp == kTmaWarp1) {
            // ================================ TMA producer ================================================
            if (lane == 0) {
                for (int j = J0; j < J1; ++j) {
                    const int n = j - J0;
                    if (n > 0) mbar_wait(bar_ek, (n - 1) & 1, abort_flag, p.wait_cycles, p.status, 10);
                    mbar_expect_tx(bar_fk, kTileBytes);
                    tma_load_4d(sbase + kOffK1, &mapK, bar_fk, 0, kh, j * kTileN, b);
                    tma_load_4d(sbase + kOffK1 + kHalfBytes, &mapK, bar_fk, 64, kh, j * kTileN, b);
                    if (n > 0) mbar_wait(bar_ev, (n - 1) & 1, abort_flag, p.wait_cycles, p.status, 11);
                    mbar_expect_tx(bar_fv, kTileBytes);
                    tma_load_4d(sbase + kOffV1, &mapV, bar_fv, 0, kh, j * kTileN, b);
                    tma_load_4d(sbase + kOffV1 + kHalfBytes, &mapV, bar_fv, 64, kh, j * kTileN, b);
                }
            }
        } else {
            // ================================ MMA issuer ==================================================
            if (lane == 0) {
                auto issue_qk = [&]() {           // S = Q K_j^T : 8 steps of 16 dims
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk) {
                        const uint32_t off = (kk >> 2) * kHalfBytes + (kk & 3) * 32;
                        mma_ss(tmem, desc_kmajor(sbase + kOffQ1 + off), desc_kmajor(sbase + kOffK1 + off), kIdescQK, kk > 0);
                    }
                    mma_commit(bar_s);
                    mma_commit(bar_ek);
                };
                mbar_wait(bar_q, 0, abort_flag, p.wait_cycles, p.status, 20);
                mbar_wait(bar_fk, 0, abort_flag, p.wait_cycles, p.status, 21);
                tc_fence_after();
                issue_qk();
                for (int j = J0; j < J1; ++j) {
                    const int n = j - J0;
                    mbar_wait(bar_fv, n & 1, abort_flag, p.wait_cycles, p.status, 22);
                    mbar_wait(bar_p, n & 1, abort_flag, p.wait_cycles, p.status, 24);
                    tc_fence_after();
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk)    // O (+)= P V_j : 8 steps of 16 keys
                        mma_ts(tmem + 128, tmem + kk * 8, desc_mnmajor(sbase + kOffV1 + kk * 16 * 128, kHalfBytes), kIdescPV,
                               (n > 0 || kk > 0) ? 1u : 0u);
                    mma_commit(bar_ev);
                    if (j + 1 < J1) {
                        mbar_wait(bar_fk, (n + 1) & 1, abort_flag, p.wait_cycles, p.status, 23);
                        tc_fence_after();
                        issue_qk();
                    }
                }
                mma_commit(bar_o);
            }
        }
    } else {
        // ================================ softmax group ================================================
        asm volatile("setmaxnreg.inc.sync.aligned.u32 200;");
        const int r = tid;                        // row within the tile
        const int slot = slot0 + r;
        const bool valid = slot < nk;
        int hi = t_row;                                                           // visible keys: lo .. hi
        int lo = (valid && p.window > 0) ? max(0, t_row - p.window + 1) : 0;
        if (p.compact && valid) {
            lo = p.window > 0 ? first_kept_at_or_after(kept, slot + 1, lo) : 0;
            hi = slot;
        }
        {   // gather the Q rows into the swizzled K-major operand layout
            const int sub = lane >> 4, cc = lane & 15;
            uint4 qv[kRounds];
            const __nv_bfloat16* qbase = p.Q + (long long)b * p.qs.b + (long long)qh * p.qs.h + cc * 8;
#pragma unroll
            for (int it = 0; it < kRounds; ++it) qv[it] = tq[it] >= 0 ? ldg16(qbase + (long long)tq[it] * p.qs.t) : zero4;
#pragma unroll
            for (int it = 0; it < kRounds; ++it)
                *reinterpret_cast<uint4*>(smem + kOffQ1 + swz(it * 8 + warp * 2 + sub, cc)) = qv[it];
            fence_proxy_async();
            mbar_arrive(bar_q);
        }
        __syncwarp();
        const uint32_t tm_s = tmem + ((uint32_t)(warp * 32) << 16);   // this warp's lanes: S / P
        const uint32_t tm_o = tm_s + 128;                             // O
        float m_ref = -INFINITY, l_run = 0.f;
        for (int j = J0; j < J1; ++j) {
            const int n = j - J0;
            mbar_wait(bar_s, n & 1, abort_flag, p.wait_cycles, p.status, 30);
            __syncwarp();
            tc_fence_after();
            softmax_tile(tm_s, tm_o, lo, hi, j * kTileN, p.scale_log2, n > 0, m_ref, l_run);
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(bar_p);
        }
        // ---- epilogue: O / l -> bf16 -> staged in the Q tile's shared memory -> the rows' token positions ----------
        mbar_wait(bar_o, 0, abort_flag, p.wait_cycles, p.status, 40);
        __syncwarp();
        tc_fence_after();
        const float inv = 1.f / l_run;
        int* trow_s = reinterpret_cast<int*>(smem + kOffK1);          // the K slot is idle by now
        trow_s[r] = t_row;
        uint8_t* stage = smem + kOffQ1 + r * 256;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            uint32_t o[32];
            tmem_ld32(tm_o + c * 32, o);
            tmem_wait_ld();
#pragma unroll
            for (int v = 0; v < 4; ++v) {
                uint4 w;
                w.x = pack_bf16(__uint_as_float(o[8 * v + 0]) * inv, __uint_as_float(o[8 * v + 1]) * inv);
                w.y = pack_bf16(__uint_as_float(o[8 * v + 2]) * inv, __uint_as_float(o[8 * v + 3]) * inv);
                w.z = pack_bf16(__uint_as_float(o[8 * v + 4]) * inv, __uint_as_float(o[8 * v + 5]) * inv);
                w.w = pack_bf16(__uint_as_float(o[8 * v + 6]) * inv, __uint_as_float(o[8 * v + 7]) * inv);
                *reinterpret_cast<uint4*>(stage + (((c * 4 + v) ^ (r & 15)) << 4)) = w;
            }
        }
        asm volatile("bar.sync 1, %0;" :: "n"(kTileM) : "memory");      // the 128 softmax threads
        const int sub = r >> 4, l16 = r & 15;                           // 8 rows per pass
#pragma unroll
        for (int pass = 0; pass < kTileM / 8; ++pass) {
            const int R = pass * 8 + sub, t_out = trow_s[R];
            if (t_out >= 0)
                *reinterpret_cast<uint4*>(Ob + (long long)t_out * p.os.t + l16 * 8) =
                    *reinterpret_cast<const uint4*>(smem + kOffQ1 + R * 256 + ((l16 ^ (R & 15)) << 4));
        }
    }
    __syncwarp();
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {   // a wait gave up: give copies and products still in flight time to land before leaving
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000ll) { }
        __syncthreads();
    }
    if (warp == kMmaWarp1) tmem_dealloc(tmem, kTmemCols1);
}

// ---- host side: tensor maps over the caller's K / V (two 64-column boxes of kTileN keys per tile) ---------
bool make_kv_map(CUtensorMap* map, const void* base, const int64_t st[3], int B, int S, int H) {
    return make_bshd_map(map, base, st, B, S, H, 2, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 64, kTileN, CU_TENSOR_MAP_SWIZZLE_128B);
}

// TF_KV_RETAINED: copy the retained tokens' K and V rows (all KV heads) to dense [B,S,Hkv,128] buffers,
// entry c of a sequence = token kept_idx[c]; entries from n_kept up to the next multiple of the key tile
// are zeroed (they are masked, but a tile may not contain NaN bit patterns: 0 * NaN would reach O).
__global__ void __launch_bounds__(256) compact_kv_kernel(const __nv_bfloat16* __restrict__ K, const __nv_bfloat16* __restrict__ V,
                                                         Strides3 ks, Strides3 vs, int S, int Hkv,
                                                         const int32_t* __restrict__ kept_idx, const int32_t* __restrict__ n_kept,
                                                         __nv_bfloat16* __restrict__ Kc, __nv_bfloat16* __restrict__ Vc) {
    grid_dependency_wait();
    const int b = blockIdx.y, nk = n_kept[b];
    const int c_end = min(S, (nk + kTileN - 1) / kTileN * kTileN);
    const int chunks = Hkv * 16;                               // 16-byte chunks per row of one tensor
    const int32_t* kept = kept_idx + (size_t)b * S;
    for (int c = blockIdx.x * 8 + (threadIdx.x >> 5); c < c_end; c += gridDim.x * 8) {
        const bool live = c < nk;
        const long long t = live ? kept[c] : 0;
        for (int q = threadIdx.x & 31; q < chunks; q += 32) {
            const int h = q >> 4, off = (q & 15) * 8;
            uint4 kv = make_uint4(0, 0, 0, 0), vv = kv;
            if (live) {
                kv = ldg16(K + (long long)b * ks.b + t * ks.t + (long long)h * ks.h + off);
                vv = ldg16(V + (long long)b * vs.b + t * vs.t + (long long)h * vs.h + off);
            }
            const size_t dst = (((size_t)b * S + c) * Hkv + h) * kHeadDim + off;
            *reinterpret_cast<uint4*>(Kc + dst) = kv;
            *reinterpret_cast<uint4*>(Vc + dst) = vv;
        }
    }
}

}  // namespace

size_t kv_compact_bytes(const tf_shape& s) {
    return 2 * ((size_t)s.batch * s.seq * s.n_kv_heads * kHeadDim * sizeof(__nv_bfloat16) + 255) / 256 * 256;
}

cudaError_t launch_attention_tc(tf_ctx* ctx, const tf_shape& s, const tf_filter_params& p,
                                const void* Q, const void* K, const void* V,
                                const int32_t* kept_idx, const int32_t* n_kept, void* O,
                                void* kv_compact, cudaStream_t st) {
    if (s.dtype != TF_BF16 || s.head_dim != kHeadDim) return cudaErrorNotSupported;
    if (s.batch == 0 || s.seq == 0) return cudaSuccess;
    const bool compact = (p.kv_visibility == TF_KV_RETAINED);
    CUtensorMap mapK, mapV;
    if (compact) {
        if (!kv_compact) return cudaErrorNotSupported;
        __nv_bfloat16* Kc = static_cast<__nv_bfloat16*>(kv_compact);
        __nv_bfloat16* Vc = reinterpret_cast<__nv_bfloat16*>(static_cast<char*>(kv_compact) + kv_compact_bytes(s) / 2);
        const int64_t dense[3] = {(int64_t)s.seq * s.n_kv_heads * kHeadDim, (int64_t)s.n_kv_heads * kHeadDim, kHeadDim};
        if (!make_kv_map(&mapK, Kc, dense, s.batch, s.seq, s.n_kv_heads) ||
            !make_kv_map(&mapV, Vc, dense, s.batch, s.seq, s.n_kv_heads))
            return cudaErrorNotSupported;
        const Strides3 ks = {s.k_stride[0], s.k_stride[1], s.k_stride[2]}, vs = {s.v_stride[0], s.v_stride[1], s.v_stride[2]};
        const unsigned gx = (unsigned)std::min<long long>(((long long)s.seq + 7) / 8, 4096);
        cudaError_t e = launch_dependent(compact_kv_kernel, dim3(gx, (unsigned)s.batch), dim3(256), 0, st,
                                         static_cast<const __nv_bfloat16*>(K), static_cast<const __nv_bfloat16*>(V), ks, vs,
                                         s.seq, s.n_kv_heads, kept_idx, n_kept, Kc, Vc);
        ctx->launches += 1;
        if (e != cudaSuccess) return e;
    } else if (!make_kv_map(&mapK, K, s.k_stride, s.batch, s.seq, s.n_kv_heads) ||
               !make_kv_map(&mapV, V, s.v_stride, s.batch, s.seq, s.n_kv_heads))
        return cudaErrorNotSupported;
    static bool attr_set_dev[kDeviceFlagSlots] = {};      // function attributes are per device
    bool& attr_set = attr_set_dev[ctx->device >= 0 && ctx->device < kDeviceFlagSlots ? ctx->device : 0];
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(attention_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             Cfg<false>::kSmemBytes);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(attention_tc_kernel<false, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     Cfg<false>::kSmemBytes);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(attention_tc_kernel<false, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     Cfg<false>::kSmemBytes);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(attention_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     Cfg<true>::kSmemBytes);
        if (e != cudaSuccess) return e;
        // The kernel moves registers from its third warpgroup to the softmax warpgroups (setmaxnreg: 168 -> 72
        // releases 128 x 96, 168 -> 216 takes 256 x 48).  An inc only receives what a dec of the same CTA
        // released and waits for it without limit, so the trade must balance: refuse to launch a build that
        // does not start at 168 registers per thread.
        // That is a defect of the build, not a property of the call: it is reported as an error of its own and
        // never answered by running another kernel.
        cudaFuncAttributes fa{};
        if (cudaFuncGetAttributes(&fa, attention_tc_kernel<false>) != cudaSuccess || fa.numRegs != 168 ||
            cudaFuncGetAttributes(&fa, attention_tc_kernel<false, 1>) != cudaSuccess || fa.numRegs != 168 ||
            cudaFuncGetAttributes(&fa, attention_tc_kernel<false, 2>) != cudaSuccess || fa.numRegs != 168 ||
            cudaFuncGetAttributes(&fa, attention_tc_kernel<true>) != cudaSuccess || fa.numRegs != 168)
            return cudaErrorInvalidDeviceFunction;
        // the single form: 256 threads at 128 registers, traded 128 x 200 + 128 x 56
        e = cudaFuncSetAttribute(attention_tc_single_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes1);
        if (e != cudaSuccess) return e;
        if (cudaFuncGetAttributes(&fa, attention_tc_single_kernel) != cudaSuccess || fa.numRegs != kRegs1)
            return cudaErrorInvalidDeviceFunction;
        attr_set = true;
    }
    TcParams tp{};
    tp.Q = static_cast<const __nv_bfloat16*>(Q);
    tp.O = static_cast<__nv_bfloat16*>(O);
    tp.qs = {s.q_stride[0], s.q_stride[1], s.q_stride[2]};
    tp.os = {s.o_stride[0], s.o_stride[1], s.o_stride[2]};
    tp.S = s.seq; tp.Hq = s.n_q_heads; tp.Hkv = s.n_kv_heads; tp.window = s.window;
    const float scale = s.softmax_scale != 0.f ? s.softmax_scale : 1.f / sqrtf((float)s.head_dim);
    tp.scale_log2 = scale * 1.4426950408889634f;
    tp.kept_idx = kept_idx; tp.n_kept = n_kept;
    tp.status = ctx->dev_status;
    tp.compact = compact ? 1 : 0;
    tp.wait_cycles = ctx_wait_cycles(ctx);
    // The shared form needs enough CTAs to fill and balance the SMs (CTAs of one head differ in length by
    // the causal triangle); below that the split form, with twice as many CTAs of half the length, wins.
    // The number of retained rows is only known on the device: the ratio gives the expected count.
    const double kept_frac = (p.select_mode == TF_SELECT_RATIO) ? 1.0 - p.prune_ratio : 1.0;
    const double ctas_shared = (double)s.batch * s.n_q_heads * ceil(s.seq * kept_frac / (kQTiles * kTileM));
    int sms = 148;
    { int dev = 0; if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev); }
    const bool single = ctx->attention_form == 3;
    const bool split = ctx->attention_form == 2 || (ctx->attention_form == 0 && ctas_shared < 1.0 * sms);
    // Grouped-query attention with an even number of query heads per KV head: the two Q tiles of a shared-form CTA are
    // the same 128 retained rows of two query heads of one group instead of 256 rows of one head; with a multiple of
    // four, the same 64 rows of four heads (two per tile): the shorter the span of positions a CTA's rows cover, the
    // fewer K/V tiles it has to visit beyond the window (or the causal triangle) itself.
    const int q_per_kv = (s.n_kv_heads > 0 && s.n_q_heads % s.n_kv_heads == 0) ? s.n_q_heads / s.n_kv_heads : 1;
    if ((ctx->attention_form == 4 && q_per_kv % 2) || (ctx->attention_form == 5 && q_per_kv % 4)) return cudaErrorNotSupported;
    const int hpt = ctx->attention_form == 4 ? 1 : ctx->attention_form == 5 ? 2     // heads per Q tile, 0 = one head per CTA
                  : (ctx->attention_form == 0 && !split) ? (q_per_kv % 4 == 0 ? 2 : q_per_kv % 2 == 0 ? 1 : 0) : 0;
    const bool heads = hpt > 0;
    const int rows_per_cta = heads ? kTileM / hpt : (split || single) ? kTileM : kQTiles * kTileM;
    tp.n_row_blocks = (s.seq + rows_per_cta - 1) / rows_per_cta;
    {
        const long long kept_est = (p.select_mode == TF_SELECT_RATIO) ? (long long)s.seq - (long long)floor(p.prune_ratio * (double)s.seq)
                                                                      : (long long)s.seq;
        const long long blocks = (std::max<long long>(kept_est, 1) + rows_per_cta - 1) / rows_per_cta;
        tp.first_pair = (int)std::min<long long>(std::max<long long>(blocks - 1, 0), tp.n_row_blocks - 1);
    }
    const long long n_bh = (long long)(heads ? s.n_q_heads / (2 * hpt) : s.n_q_heads) * s.batch;
    const long long n_ctas = (long long)tp.n_row_blocks * n_bh;
    {
        // Groups of (batch, head) pairs.  Heaviest-first over ALL heads balances best and costs nothing while all of K
        // and V stays in L2 (c4: 555 -> 526 us).  Once the K and V of the heads that run together exceed L2, every CTA
        // streams its keys from HBM (3.9 KB per MFLOP of tile products): in short loops the balance still wins
        // (c3: 405 -> 372 us), under the power cap of a long run the HBM traffic lowers the clock and loses
        // (425 -> 445 us).  So a group is as many pairs as keep their K and V within kL2Budget, in equal groups
        // (c3: 5 groups of 32 heads, 438 -> 422 us in long loops, 430 -> 397 in short ones).  A window makes the row
        // blocks equally long, so there is nothing to balance and the row blocks of a pair stay together (c5: every
        // larger group measured 2-12 % slower).  A grid of a few CTAs per SM is balanced over all heads whatever the size.
        constexpr double kL2Budget = 72e6;
        const double kv_all = 2.0 * s.batch * (double)s.seq * s.n_kv_heads * kHeadDim * sizeof(__nv_bfloat16);
        const double kv_per_bh = kv_all / (double)std::max<long long>(n_bh, 1);
        const bool windowed = s.window > 0 && (long long)s.window + 1024 < s.seq;
        long long g = windowed ? 1 : std::max<long long>((long long)(kL2Budget / kv_per_bh), 1);
        if (kv_all <= kL2Budget || ctas_shared < 6.0 * sms) g = n_bh;
        g = std::min<long long>(g, std::max<long long>(n_bh, 1));
        const long long n_groups = (std::max<long long>(n_bh, 1) + g - 1) / g;      // equal groups, not a small last one
        g = (std::max<long long>(n_bh, 1) + n_groups - 1) / n_groups;
        tp.bh_group = (int)std::min<long long>(std::max<long long>(g, 1), std::max<long long>(n_bh, 1));
    }
    if (n_ctas > 0x7fffffffll) return cudaErrorInvalidValue;
    cudaError_t e;
    if (single) e = launch_dependent(attention_tc_single_kernel, dim3((unsigned)n_ctas), dim3(kThreads1), kSmemBytes1, st, tp, mapK, mapV);
    else if (hpt == 2) e = launch_dependent(attention_tc_kernel<false, 2>, dim3((unsigned)n_ctas), dim3(kThreads), Cfg<false>::kSmemBytes, st, tp, mapK, mapV);
    else if (hpt == 1) e = launch_dependent(attention_tc_kernel<false, 1>, dim3((unsigned)n_ctas), dim3(kThreads), Cfg<false>::kSmemBytes, st, tp, mapK, mapV);
    else if (split) e = launch_dependent(attention_tc_kernel<true>, dim3((unsigned)n_ctas), dim3(kThreads), Cfg<true>::kSmemBytes, st, tp, mapK, mapV);
    else       e = launch_dependent(attention_tc_kernel<false>, dim3((unsigned)n_ctas), dim3(kThreads), Cfg<false>::kSmemBytes, st, tp, mapK, mapV);
    ctx->launches += 1;
    ctx->last_attention_kernel = single ? TF_KERNEL_ATTN_TC_SINGLE : hpt == 2 ? TF_KERNEL_ATTN_TC_HEAD_QUAD : hpt == 1 ? TF_KERNEL_ATTN_TC_HEAD_PAIR
                                        : split ? TF_KERNEL_ATTN_TC_SPLIT : TF_KERNEL_ATTN_TC_SHARED;
    return e;
}

}  // namespace tf
