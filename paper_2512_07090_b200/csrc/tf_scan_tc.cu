// Steps a1+a2 for bf16 tensors with running-sum anchors, rearranged so that the CUDA cores touch
// O(tokens) values per tile instead of O(tokens x dims):
//
// For a tile X of 128 tokens of one (sequence, KV head) and the sum C of everything before it,
//   <x_i, P_i>   = <x_i, C> + sum_{j<i} G_ij        with  G = X X^T  (128 x 128)
//   ||x_i||^2    = G_ii
//   ||P_{i+1}||^2 = ||P_i||^2 + 2 <x_i, P_i> + G_ii  (a prefix sum over the tile, seeded with ||C||^2)
//   column sums of X (the tile's aggregate for the look-back) = X^T 1
// G, X^T 1 and X C are small dense products; they run on the tensor cores (tcgen05, operands in
// shared memory exactly as TMA delivers them, accumulators in TMEM), C entering as three bf16
// terms c1+c2+c3 so that the fp32 carry loses nothing.  Thread i then owns token row i: it adds
// the part of row i of G left of the diagonal, joins a block-wide prefix sum and writes the two
// cosines.  The fp32 instruction stream per (token, head) drops from ~130 to ~20 warp
// instructions, which is what kept the plain kernel from reaching the memory roofline.
//
// EMA anchors (Eq. 1: anchor <- g anchor + (1-g) x, compared before it is updated) take the same products with
// weights on the CUDA-core side.  With A0 the anchor before the tile:
//   <x_i, A_i>    = g^i <x_i, A0> + (1-g) sum_{j<i} g^(i-1-j) G_ij     (row sums become Horner recurrences in g)
//   ||A_{i+1}||^2 = g^2 ||A_i||^2 + 2 g (1-g) <x_i, A_i> + (1-g)^2 G_ii   (a prefix scan with ratio g^2)
//   A_128         = g^128 A0 + (1-g) sum_j g^(127-j) x_j                 (the "ones" row of the small operand becomes
//                                                                         three rows, 5-7, of bf16 terms of these weights)
//
// One CTA (128 threads) per (tile, tensor): K and V are independent here, and the smaller footprint
// (32 KiB of rows, 64 TMEM columns, reused in turn for X^T 1, the two halves of G and X C) lets six CTAs
// share an SM, so that the loads of some overlap the arithmetic of others.  Carries travel through tagged
// records with the same fixed-association look-back as the plain kernel (see tf_scan.cu); a record is 128
// 8-byte packets {value, tag}.  All waits are bounded.
#include <algorithm>
#include <utility>

#include "tf_ptx.cuh"

namespace tf {
namespace {

constexpr int kGT = 128;                       // tokens per tile
constexpr int kHalf = 128 * 128;               // one [128 rows][128 B] swizzled block
constexpr int kXBytes = 2 * kHalf;             // one tensor's tile
constexpr int kBtBytes = 2 * 16 * 128;         // small B operand: [16 rows][128 elements], two 64-element blocks
constexpr int kGramAnchorEvery = 4;             // a prefix record every 4th chunk: at most 4 aggregates + 1 prefix per look-back

// instruction descriptors: D fp32, A/B bf16, M = 128
constexpr uint32_t idesc(uint32_t n, bool a_mn) { return idesc_bf16(n, a_mn, false); }
constexpr uint32_t kIdescAgg = idesc(16, true);    // X^T Bt^T  (A = X taken MN-major: rows = dims)
constexpr uint32_t kIdescU = idesc(16, false);     // X Bt^T

// byte offset of element (row n, index k) of the small B operand (K-major, 128-byte swizzle)
__device__ __forceinline__ uint32_t bt_off(int n, int k) {
    return (uint32_t)((k >> 6) * (16 * 128) + n * 128 + ((((k & 63) >> 3) ^ (n & 7)) << 4) + (k & 7) * 2);
}
__device__ __forceinline__ unsigned short bf16_bits(float x) { return __bfloat16_as_ushort(__float2bfloat16_rn(x)); }


// ---- the two anchor forms: what differs between running sums and EMA anchors on the CUDA-core side ---------------
// g^k for a small non-negative integer k (square-and-multiply: a few roundings, no transcendental)
__device__ __forceinline__ float powi(float g, int k) {
    float r = 1.f, b = g;
    for (; k > 0; k >>= 1) {
        if (k & 1) r *= b;
        b *= b;
    }
    return r;
}
template <bool EMA> struct Anchor;
template <> struct Anchor<false> {
    __device__ __forceinline__ Anchor(float, int, int) {}
    // thread i's row of G: a 32-column block wholly left of the diagonal / the block that holds the diagonal
    __device__ __forceinline__ void full_block(const uint32_t* g, float& acc) const {
        float s4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int e = 0; e < 32; ++e) s4[e & 3] += __uint_as_float(g[e]);
        acc += (s4[0] + s4[1]) + (s4[2] + s4[3]);
    }
    __device__ __forceinline__ void diag_block(const uint32_t* g, int lane, float& part, float& g_diag) const {
#pragma unroll
        for (int e = 0; e < 32; ++e) {
            const float v = __uint_as_float(g[e]);
            part += (e < lane) ? v : 0.f;
            g_diag = (e == lane) ? v : g_diag;
        }
    }
    __device__ __forceinline__ float dot(float u, float acc, float part) const { return u + (acc + part); }   // <x_i, P_i>
    __device__ __forceinline__ float norm_step(float d, float g_diag) const { return fmaf(2.f, d, g_diag); } // ||P_{i+1}||^2 - ||P_i||^2
    __device__ __forceinline__ float look_back(float A, float agg) const { return A + agg; }
    __device__ __forceinline__ float carry_of(float prefix, float A, int) const { return prefix + A; }
    __device__ __forceinline__ float sum_after(float carry, float agg, int) const { return carry + agg; }
    __device__ __forceinline__ float agg_of(const uint32_t* r) const { return __uint_as_float(r[6]); }
    // the block-wide exclusive prefix of the norm steps, seeded with n0; red: [4 warps] stride 2; sync: a barrier over the 128 threads
    template <typename Sync>
    __device__ __forceinline__ float norm_before(float b, float n0, int warp, int lane, volatile float* red, Sync sync) const {
        float incl = b;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const float n = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += n;
        }
        if (lane == 31) red[warp * 2] = incl;
        sync();
        float off = n0;
        for (int w2 = 0; w2 < warp; ++w2) off += red[w2 * 2];
        return off + (incl - b);
    }
};
template <> struct Anchor<true> {
    float g, w, g8, g32, g128, pw_lane, pw_row, q32, q_lane, qs[5];
    __device__ __forceinline__ Anchor(float gamma, int warp, int lane) {
        g = gamma; w = 1.f - gamma;
        g8 = powi(g, 8); g32 = powi(g, 32); g128 = powi(g, 128);
        pw_lane = powi(g, lane); pw_row = powi(g, 32 * warp + lane);
        q32 = powi(g, 64); q_lane = powi(g, 2 * lane);
#pragma unroll
        for (int k = 0; k < 5; ++k) qs[k] = powi(g, 2 << k);
    }
    // sum_e G[e] g^(31-e), then acc <- acc g^32 + that: after the blocks left of the diagonal, acc = sum_j g^(32 W - 1 - j) G_ij
    __device__ __forceinline__ void full_block(const uint32_t* gr, float& acc) const {
        float h[4];
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            h[c] = __uint_as_float(gr[8 * c]);
#pragma unroll
            for (int e = 1; e < 8; ++e) h[c] = fmaf(h[c], g, __uint_as_float(gr[8 * c + e]));
        }
        const float r = fmaf(fmaf(fmaf(h[0], g8, h[1]), g8, h[2]), g8, h[3]);
        acc = fmaf(acc, g32, r);
    }
    // sum_{e < lane} G[e] g^(lane-1-e)
    __device__ __forceinline__ void diag_block(const uint32_t* gr, int lane, float& part, float& g_diag) const {
#pragma unroll
        for (int e = 0; e < 32; ++e) {
            const float v = __uint_as_float(gr[e]);
            part = (e < lane) ? fmaf(part, g, v) : part;
            g_diag = (e == lane) ? v : g_diag;
        }
    }
    __device__ __forceinline__ float dot(float u, float acc, float part) const { return fmaf(pw_row, u, w * fmaf(pw_lane, acc, part)); }
    __device__ __forceinline__ float norm_step(float d, float g_diag) const { return fmaf(2.f * g * w, d, w * w * g_diag); }
    __device__ __forceinline__ float look_back(float A, float agg) const { return fmaf(A, g128, agg); }
    __device__ __forceinline__ float carry_of(float prefix, float A, int chunks) const {
        float f = g128;
        for (int m = 1; m < chunks; ++m) f *= g128;
        return fmaf(f, prefix, A);
    }
    __device__ __forceinline__ float sum_after(float carry, float agg, int valid) const {
        return fmaf(valid == kGT ? g128 : powi(g, valid), carry, agg);
    }
    __device__ __forceinline__ float agg_of(const uint32_t* r) const {
        return (__uint_as_float(r[5]) + __uint_as_float(r[6])) + __uint_as_float(r[7]);
    }
    template <typename Sync>
    __device__ __forceinline__ float norm_before(float b, float n0, int warp, int lane, volatile float* red, Sync sync) const {
        float incl = b;                                  // sum_{j <= i, same warp} q^(i-j) b_j, q = g^2
#pragma unroll
        for (int k = 0; k < 5; ++k) {
            const float n = __shfl_up_sync(0xffffffffu, incl, 1 << k);
            if (lane >= (1 << k)) incl = fmaf(qs[k], n, incl);
        }
        if (lane == 31) red[warp * 2] = incl;
        float excl = __shfl_up_sync(0xffffffffu, incl, 1);
        if (lane == 0) excl = 0.f;
        sync();
        float cw = n0;                                   // ||A||^2 before this warp's first token
        for (int w2 = 0; w2 < warp; ++w2) cw = fmaf(cw, q32, red[w2 * 2]);
        return fmaf(q_lane, cw, excl);
    }
};
// cosine of x_i to its anchor from d = <x_i, anchor sum>, xx = ||x_i||^2, pp = ||anchor sum||^2; the running-sum anchor
// is the sum over cnt tokens divided by cnt (the division cancels unless a norm falls under its clamp), the EMA anchor is
// the sum itself
template <bool EMA>
__device__ __forceinline__ float anchor_cosine(float d, float xx, float pp, long long cnt) {
    if (cnt <= 0) return 0.f;
    const float fc = EMA ? 1.f : (float)cnt, lim = kNormEps * kNormEps;
    if (xx > lim && pp > lim * fc * fc) return d * rsqrtf(xx) * rsqrtf(pp);
    const float sc = 1.f / fc;
    return (d * sc) / (fmaxf(sqrtf(xx), kNormEps) * fmaxf(sqrtf(fmaxf(pp, 0.f)) * sc, kNormEps));
}
// the weight of token t of a tile with `valid` tokens in the tile's aggregate, as three bf16 terms
template <bool EMA>
__device__ __forceinline__ void agg_weight_terms(float gamma, int t, int valid, unsigned short out[3]) {
    if (!EMA) { out[0] = 0x3f80; out[1] = 0; out[2] = 0; return; }      // 1, 0, 0
    float wv = t < valid ? (1.f - gamma) * powi(gamma, valid - 1 - t) : 0.f;
#pragma unroll
    for (int n = 0; n < 3; ++n) {
        out[n] = bf16_bits(wv);
        wv -= __uint_as_float((uint32_t)out[n] << 16);
    }
}

__device__ __forceinline__ bool wait_bar(uint32_t bar, uint32_t parity, volatile int* abort_flag, long long budget_cycles,
                                         DevStatus* status, unsigned long long where) {
    return mbar_wait_bounded(bar, parity, abort_flag, budget_cycles, status, where);
}

// One CTA per (tile, tensor): 32 KiB of rows, 64 TMEM columns, so six CTAs share an SM and their loads
// overlap one another's arithmetic.
constexpr int kT1OffX = 0, kT1OffBt = kXBytes, kT1OffMisc = kT1OffBt + kBtBytes;
constexpr int kT1Smem = kT1OffMisc + 256;          // the dynamic segment must start 1024-byte aligned (checked)
constexpr uint32_t kT1TmemCols = 64;
constexpr uint32_t kIdescG64 = idesc(64, false);   // 64 columns of G at a time

struct Gram1Params {
    int S, H, n_chains, n_chunks;
    int incl;
    float gamma;                 // EMA anchors only
    const float* sum_in[2]; const long long* count_in;
    float* sum_out[2];
    float* sim[2];
    uint2* agg_rec[2]; uint2* prefix_rec[2];
    DevStatus* status;
    int max_polls;               // bounded waits: polls of one look-back packet ...
    long long wait_cycles;       // ... and clock cycles of one mbarrier wait
    unsigned int* counters;      // {ticket, finished}: see ScanScratch
    unsigned int n_work;         // (tile, tensor) pairs
};

template <bool EMA>
__global__ void __launch_bounds__(128, 6)
kv_stats_gram1_kernel(const Gram1Params p, const __grid_constant__ CUtensorMap mapK, const __grid_constant__ CUtensorMap mapV) {
    extern __shared__ uint8_t smem[];
    const uint32_t sbase = smem_u32(smem);
    if (sbase & 1023u) {   // the swizzled operand layout needs it; nothing has been started yet
        if (threadIdx.x == 0) {
            report_error(p.status, TF_ERR_TIMEOUT, 199);
            grid_dependency_wait();
            scan_draw_ticket(p.counters);
            scan_leave(p.counters, gridDim.x);
        }
        return;
    }
    const uint32_t bar_tma = sbase + kT1OffMisc, bar_mma = bar_tma + 8;
    volatile unsigned int* s_ticket = reinterpret_cast<volatile unsigned int*>(smem + kT1OffMisc + 96);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + kT1OffMisc + 16);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + kT1OffMisc + 24);
    float* red = reinterpret_cast<float*>(smem + kT1OffMisc + 32);     // [4 warps][2] block reduction / scan scratch

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        mbar_init(bar_tma, 1);
        mbar_init(bar_mma, 1);
        *abort_flag = 0;
        mbar_fence_init();
    }
    // small B operand: rows 0-2 will take the three bf16 terms of the carry, row 6 is all ones, the rest 0
    *reinterpret_cast<uint4*>(smem + kT1OffBt + tid * 32) = make_uint4(0, 0, 0, 0);
    *reinterpret_cast<uint4*>(smem + kT1OffBt + tid * 32 + 16) = make_uint4(0, 0, 0, 0);
    __syncthreads();
    if (!EMA) *reinterpret_cast<unsigned short*>(smem + kT1OffBt + bt_off(6, tid)) = 0x3f80;
    const Anchor<EMA> an(p.gamma, warp, lane);
    if (warp == 1) tmem_alloc(smem_u32(tmem_slot), kT1TmemCols);
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    const uint32_t tm_lane = tmem + ((uint32_t)(warp * 32) << 16);
    grid_dependency_wait();   // launched so that the set-up above overlaps the tail of the kernel before it on the stream

    // Work goes by ticket, chunk index slowest (K and V of a tile side by side): the records a tile waits for belong
    // to tickets drawn before its own, by CTAs that are running, whatever order the CTAs were started in.
    if (tid == 0) {
        s_ticket[1] = scan_launch_tag(p.counters);
        const unsigned int t = scan_draw_ticket(p.counters);
        scan_leave(p.counters, gridDim.x);     // one ticket per CTA
        *s_ticket = t;
        if (t < p.n_work) {
            const unsigned int tile0 = t >> 1;
            const int c0 = (int)(tile0 / (unsigned)p.n_chains), chain0 = (int)(tile0 % (unsigned)p.n_chains);
            const CUtensorMap* map = (t & 1) ? &mapV : &mapK;
            mbar_expect_tx(bar_tma, kXBytes);
            tma_load_4d(sbase + kT1OffX, map, bar_tma, 0, chain0 % p.H, c0 * kGT, chain0 / p.H);
            tma_load_4d(sbase + kT1OffX + kHalf, map, bar_tma, 64, chain0 % p.H, c0 * kGT, chain0 / p.H);
        }
    }
    __syncthreads();
    const unsigned int ticket = s_ticket[0], epoch = s_ticket[1];
    if (ticket >= p.n_work) {                  // cannot happen while the counters are intact; never index records with it
        tc_fence_before();
        __syncthreads();
        if (warp == 1) tmem_dealloc(tmem, kT1TmemCols);
        return;
    }
    const int x = ticket & 1;
    const unsigned int tile = ticket >> 1;
    const int c = (int)(tile / (unsigned)p.n_chains), chain = (int)(tile % (unsigned)p.n_chains);
    const int b = chain / p.H, h = chain % p.H;
    const uint32_t xa = sbase + kT1OffX, bt = sbase + kT1OffBt;
    uint2* agg_rec = p.agg_rec[x];
    uint2* prefix_rec = p.prefix_rec[x];

    // look-back requests go out while the tile is in flight
    const bool has_prev = c > 0;
    const int a0 = has_prev ? ((c - 1) / kGramAnchorEvery) * kGramAnchorEvery : 0;
    const uint2* prec = prefix_rec + ((size_t)(a0 / kGramAnchorEvery) * p.n_chains + chain) * kHeadDim + tid;
    uint2 pfirst = make_uint2(0, 0), afirst[kGramAnchorEvery];
    const uint2* arec = agg_rec + ((size_t)a0 * p.n_chains + chain) * kHeadDim + tid;      // chunk a0 + u: u n_chains records on
    const size_t astride = (size_t)p.n_chains * kHeadDim;
    if (has_prev) {
        pfirst = ld_packet2(prec);
#pragma unroll
        for (int u = 0; u < kGramAnchorEvery; ++u)
            if (a0 + u < c) afirst[u] = ld_packet2(arec + u * astride);
    }

    const int valid = min(kGT, p.S - c * kGT);       // tokens in this tile
    if (EMA) {      // the aggregate's weights (rows 5-7 of the small operand, element = token) depend on the tile's length
        unsigned short wt[3];
        agg_weight_terms<EMA>(p.gamma, tid, valid, wt);
#pragma unroll
        for (int n = 0; n < 3; ++n) *reinterpret_cast<unsigned short*>(smem + kT1OffBt + bt_off(5 + n, tid)) = wt[n];
        fence_proxy_async();
        __syncthreads();
    }
    uint32_t mma_phase = 0;
    wait_bar(bar_tma, 0, abort_flag, p.wait_cycles, p.status, 100);

    // ---- 1. column sums: (X^T Bt^T)[d][6] = sum_t X[t][d]; two interleaved accumulator chains ------------
    if (tid == 0) {
        tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < 8; ++kk)         // 16 tokens per step
            mma_ss(tmem + 16 * (kk & 1), desc_mnmajor(xa + kk * 16 * 128, kHalf),
                   desc_kmajor(bt + (kk >> 2) * (16 * 128) + (kk & 3) * 32), kIdescAgg, kk > 1);
        mma_commit(bar_mma);
    }
    wait_bar(bar_mma, mma_phase, abort_flag, p.wait_cycles, p.status, 101); mma_phase ^= 1;
    tc_fence_after();
    float agg;
    {
        uint32_t r0[8], r1[8];
        tmem_ld8(tm_lane, r0);
        tmem_ld8(tm_lane + 16, r1);
        tmem_wait_ld();
        agg = an.agg_of(r0) + an.agg_of(r1);
    }
    if (c + 1 < p.n_chunks) st_packet2(agg_rec + (size_t)tile * kHeadDim + tid, agg, epoch);
    tc_fence_before();
    __syncthreads();

    // ---- carry from earlier chunks (thread = dim).  A tile that publishes a prefix (every 8th chunk) does this
    // before its Gram matrix: its prefix depends on older tiles only, and the seven tiles after it wait for it.
    float carry = 0.f;
    auto resolve_carry = [&]() {
        if (c == 0) {
            if (p.sum_in[x]) carry = p.sum_in[x][(size_t)chain * kHeadDim + tid];
        } else {
            float A = 0.f;
#pragma unroll
            for (int u = 0; u < kGramAnchorEvery; ++u)       // requested while the tile was in flight
                if (a0 + u < c) A = an.look_back(A, wait_packet2(arec + u * astride, afirst[u], epoch, p.max_polls, p.status, tile));
            carry = an.carry_of(wait_packet2(prec, pfirst, epoch, p.max_polls, p.status, tile), A, c - a0);
        }
        if (c % kGramAnchorEvery == 0 && c + 1 < p.n_chunks)
            st_packet2(prefix_rec + ((size_t)(c / kGramAnchorEvery) * p.n_chains + chain) * kHeadDim + tid, carry, epoch);
        if (c + 1 == p.n_chunks && p.sum_out[x]) p.sum_out[x][(size_t)chain * kHeadDim + tid] = an.sum_after(carry, agg, valid);
    };
    const bool publishes_prefix = (c % kGramAnchorEvery == 0);
    if (publishes_prefix) resolve_carry();

    // ---- 2. G = X X^T, 64 columns at a time; thread i adds row i left of the diagonal ---------------------
    float r_acc = 0.f, r_part = 0.f, g_diag = 0.f;
#pragma unroll
    for (int hh = 0; hh < 2; ++hh) {
        if (tid == 0) {
            tc_fence_after();
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) {   // 16 dims per step; B = rows 64 hh .. 64 hh + 63 of the same tile
                const uint32_t off = (kk >> 2) * kHalf + (kk & 3) * 32;
                mma_ss(tmem, desc_kmajor(xa + off), desc_kmajor(xa + hh * (64 * 128) + off), kIdescG64, kk > 0);
            }
            mma_commit(bar_mma);
        }
        wait_bar(bar_mma, mma_phase, abort_flag, p.wait_cycles, p.status, 102 + hh); mma_phase ^= 1;
        tc_fence_after();
#pragma unroll
        for (int lc = 0; lc < 2; ++lc) {
            const int cb = 2 * hh + lc;               // 32-column block of G (warp-uniform comparisons)
            if (cb > warp) continue;
            uint32_t g[32];
            tmem_ld32(tm_lane + lc * 32, g);
            tmem_wait_ld();
            if (cb < warp) an.full_block(g, r_acc);
            else an.diag_block(g, lane, r_part, g_diag);
        }
        tc_fence_before();
        __syncthreads();
    }
    if (!publishes_prefix) resolve_carry();

    // ---- 3. u = X C: the carry goes into rows 0-2 of the small operand as c1 + c2 + c3 (bf16 each) ---------
    {
        float cr = carry;
#pragma unroll
        for (int n = 0; n < 3; ++n) {
            const unsigned short hb = bf16_bits(cr);
            *reinterpret_cast<unsigned short*>(smem + kT1OffBt + bt_off(n, tid)) = hb;
            cr -= __uint_as_float((uint32_t)hb << 16);
        }
    }
    float c2 = warp_sum(carry * carry);            // ||C||^2 (block sum over dims)
    if (lane == 0) red[warp * 2] = c2;
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    c2 = (red[0] + red[2]) + (red[4] + red[6]);
    if (tid == 0) {
        tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < 8; ++kk)             // 16 dims per step; two interleaved accumulator chains
            mma_ss(tmem + 16 * (kk & 1), desc_kmajor(xa + (kk >> 2) * kHalf + (kk & 3) * 32),
                   desc_kmajor(bt + (kk >> 2) * (16 * 128) + (kk & 3) * 32), kIdescU, kk > 1);
        mma_commit(bar_mma);
    }
    wait_bar(bar_mma, mma_phase, abort_flag, p.wait_cycles, p.status, 104); mma_phase ^= 1;
    tc_fence_after();
    float d;
    {
        uint32_t r0[8], r1[8];
        tmem_ld8(tm_lane, r0);
        tmem_ld8(tm_lane + 16, r1);
        tmem_wait_ld();
        auto f = [](uint32_t a, uint32_t b2) { return __uint_as_float(a) + __uint_as_float(b2); };
        d = an.dot((f(r0[0], r1[0]) + f(r0[1], r1[1])) + f(r0[2], r1[2]), r_acc, r_part);   // <x_i, anchor before token i>
    }

    // ---- 4. ||anchor||^2 before each token by a block-wide prefix scan of the norm steps, then the cosine ----------
    const float bi = an.norm_step(d, g_diag);
    float pp = an.norm_before(bi, c2, warp, lane, red + 1, [] { __syncthreads(); });
    const int t_tok = c * kGT + tid;
    if (t_tok < p.S) {
        if (p.incl) { d += g_diag; pp += bi; }
        const long long cnt = (p.count_in ? p.count_in[b] : 0ll) + t_tok + (p.incl ? 1 : 0);
        p.sim[x][((size_t)b * p.S + t_tok) * p.H + h] = anchor_cosine<EMA>(d, g_diag, pp, cnt);
    }

    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000ll) { }
        __syncthreads();
    }
    if (warp == 1) tmem_dealloc(tmem, kT1TmemCols);
}


// ---------------------------------------------------------------------------------------------------------
// Persistent form: one CTA per SM with six workers of 128 threads; every worker takes tiles from an atomic
// ticket (chunk index slowest, so the records a tile waits for belong to tickets drawn before its own) and
// runs the sequence above on its own 36 KiB of shared memory and its own 80 TMEM columns.  What it changes:
//  * barriers, the small operand and TMEM are set up once per SM instead of once per tile;
//  * the tensor pipe takes ~53 cycles for any M=128 product of up to 80 columns, and with six tiles in flight
//    that pipe, not HBM, is what the one-tile kernel saturates.  Here the small operand lies directly behind
//    each 64-dim block of the tile, so that rows 64..143 of the block are "rows 64-127 of X, then c1 c2 c3":
//    the second half of G and X C are ONE product of 80 columns (24 products per tile instead of 32);
//  * X^T 1 and the first half of G are issued together, the look-back loads go out under them, and the next
//    tile's TMA load starts as soon as the last product has read the current one, under the scan and cosine.
// ---------------------------------------------------------------------------------------------------------
constexpr int kPWorkers = 6;
constexpr int kPThreads = kPWorkers * 128;
constexpr int kPBlock = kHalf + 16 * 128;                            // [128 tile rows + 16 small-operand rows][128 B]
constexpr int kPWorkerBytes = 2 * kPBlock;                           // 36 KiB: dims 0-63, dims 64-127
constexpr int kPOffMisc = kPWorkers * kPWorkerBytes;
constexpr int kPMiscPerWorker = 96;                                  // 3 mbarriers, next ticket, scan scratch
constexpr int kPSmem = kPOffMisc + kPWorkers * kPMiscPerWorker + 64;
constexpr uint32_t kPTmemCols = 512;                                 // worker w: columns 80 w .. 80 w + 79
constexpr uint32_t kPNoTile = 0xffffffffu;
constexpr uint32_t kIdescG80 = idesc(80, false);
constexpr int kPLookBack = kGramAnchorEvery - 1;                     // aggregates between a prefix record and a tile

struct GramPParams {
    Gram1Params g;               // g.n_work counts (tile, tensor) pairs
};

// Eight products of one accumulation chain.  The operand descriptors differ only in the 14-bit address field of
// their low word, so the issuing thread adds compile-time offsets (units of 16 bytes) to two precomputed low
// words instead of rebuilding 64-bit descriptors per product: issue is on the critical path of every tile.
template <uint32_t A_OFF, uint32_t B_OFF, bool ACC>
__device__ __forceinline__ void mma_step(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t b_hi, uint32_t id) {
    asm volatile("{\n.reg .pred p;\n.reg .b32 ta, tb;\n.reg .b64 da, db;\n"
                 "setp.ne.b32 p, %6, 0;\n"
                 "add.u32 ta, %1, %7;\nadd.u32 tb, %3, %8;\n"
                 "mov.b64 da, {ta, %2};\nmov.b64 db, {tb, %4};\n"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %5, p;\n}"
                 :: "r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(id), "n"(ACC ? 1 : 0), "n"(A_OFF), "n"(B_OFF)
                 : "memory");
}
__host__ __device__ constexpr uint32_t kmaj_step(int kk, int block_bytes) { return (uint32_t)(((kk >> 2) * block_bytes + (kk & 3) * 32) >> 4); }
template <int BLOCK, bool A_MN, int... KK>
__device__ __forceinline__ void mma_burst(std::integer_sequence<int, KK...>, uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi,
                                          uint32_t b_lo, uint32_t b_hi, uint32_t id) {
    (mma_step<(A_MN ? (uint32_t)(KK * 16 * 128 >> 4) : kmaj_step(KK, BLOCK)), kmaj_step(KK, BLOCK), (KK > 0)>(d_tmem, a_lo, a_hi, b_lo, b_hi, id), ...);
}
__device__ __forceinline__ bool wait_bar_parked(uint32_t bar, uint32_t parity, volatile int* abort_flag, long long budget_cycles,
                                                DevStatus* status, unsigned long long where) {
    return mbar_wait_parked(bar, parity, abort_flag, budget_cycles, status, where);
}
__device__ __forceinline__ void worker_sync(int w) { asm volatile("bar.sync %0, 128;" :: "r"(w + 1) : "memory"); }
// byte offset, from the worker's base, of element (row n, index k) of the small operand
__device__ __forceinline__ uint32_t pbt_off(int n, int k) {
    return (uint32_t)((k >> 6) * kPBlock + kHalf + n * 128 + ((((k & 63) >> 3) ^ (n & 7)) << 4) + (k & 7) * 2);
}

template <bool EMA>
__global__ void __launch_bounds__(kPThreads, 1)
kv_stats_gram_persistent_kernel(const GramPParams pp, const __grid_constant__ CUtensorMap mapK,
                                const __grid_constant__ CUtensorMap mapV) {
    extern __shared__ uint8_t smem[];
    const Gram1Params& p = pp.g;
    const uint32_t sbase = smem_u32(smem);
    if (sbase & 1023u) {
        if (threadIdx.x == 0) {
            report_error(p.status, TF_ERR_TIMEOUT, 299);
            grid_dependency_wait();
            scan_leave(p.counters, gridDim.x);
        }
        return;
    }
    const int tid = threadIdx.x & 127, w = threadIdx.x >> 7, warp = tid >> 5, lane = tid & 31;
    uint8_t* misc = smem + kPOffMisc + w * kPMiscPerWorker;
    const uint32_t bar_tma = smem_u32(misc), bar_small = bar_tma + 8, bar_g = bar_tma + 16;
    volatile unsigned int* s_next = reinterpret_cast<volatile unsigned int*>(misc + 32);   // next tile: {chunk, chain, sequence, head | tensor << 30}
    float* red = reinterpret_cast<float*>(misc + 48);                 // [4 warps][2]
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + kPOffMisc + kPWorkers * kPMiscPerWorker);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    uint8_t* my = smem + w * kPWorkerBytes;
    const uint32_t xa = sbase + w * kPWorkerBytes;

    if (tid == 0) {
        mbar_init(bar_tma, 1);
        mbar_init(bar_small, 1);
        mbar_init(bar_g, 1);
        if (w == 0) *abort_flag = 0;
        mbar_fence_init();
    }
    // small operand (16 rows behind each 64-dim block): rows 0-2 take the carry, row 6 is all ones, the rest 0
    {
        uint8_t* dst = my + (tid >> 6) * kPBlock + kHalf + (tid & 63) * 32;
        *reinterpret_cast<uint4*>(dst) = make_uint4(0, 0, 0, 0);
        *reinterpret_cast<uint4*>(dst + 16) = make_uint4(0, 0, 0, 0);
    }
    __syncthreads();
    const Anchor<EMA> an(p.gamma, warp, lane);
    int w_valid = kGT;                // the tile length the aggregate's weights (rows 5-7, element = token) are written for
    auto write_agg_weights = [&](int valid) {
        unsigned short wt[3];
        agg_weight_terms<EMA>(p.gamma, tid, valid, wt);
        if (EMA) {
#pragma unroll
            for (int n = 0; n < 3; ++n) *reinterpret_cast<unsigned short*>(my + pbt_off(5 + n, tid)) = wt[n];
        } else {
            *reinterpret_cast<unsigned short*>(my + pbt_off(6, tid)) = wt[0];
        }
    };
    write_agg_weights(kGT);
    if (threadIdx.x < 32) tmem_alloc(smem_u32(tmem_slot), kPTmemCols);
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    const uint32_t tm_g = tmem + 80u * w, tm_s = tm_g + 64u;                       // G half / small product
    const uint32_t lane_off = (uint32_t)(warp * 32) << 16;
    // operand descriptor words (see desc_kmajor / desc_mnmajor): address field of this worker's tile, the two
    // leading-dimension fields, and the high word (8-row groups 1024 B apart, version 1, 128-byte swizzle)
    const uint32_t x_lo = (xa & 0x3ffffu) >> 4;
    constexpr uint32_t dlo_k = 1u << 16, dlo_mn = (uint32_t)(kPBlock >> 4) << 16;
    constexpr uint32_t dhi = (uint32_t)(1024 >> 4) | (1u << 14) | (2u << 29);
    constexpr std::make_integer_sequence<int, 8> k8{};

    // worker thread 0 only: decodes ticket t for everyone (the divisions are done once, off the critical path),
    // leaves the result in shared memory and starts the tile's load
    auto announce_and_load = [&](unsigned int t) {
        if (t == kPNoTile) {
            s_next[0] = kPNoTile;
            return;
        }
        const unsigned int tile = t >> 1;
        const unsigned int c = tile / (unsigned)p.n_chains, chain = tile - c * (unsigned)p.n_chains;
        const unsigned int b = chain / (unsigned)p.H, h = chain - b * (unsigned)p.H;
        s_next[0] = c; s_next[1] = chain; s_next[2] = b; s_next[3] = h | ((t & 1u) << 30);
        const CUtensorMap* map = (t & 1) ? &mapV : &mapK;
        mbar_expect_tx(bar_tma, kXBytes);
        tma_load_4d(xa, map, bar_tma, 0, (int)h, (int)c * kGT, (int)b);
        tma_load_4d(xa + kPBlock, map, bar_tma, 64, (int)h, (int)c * kGT, (int)b);
    };
    auto draw = [&]() -> unsigned int {
        const unsigned int t = scan_draw_ticket(p.counters);
        return t < p.n_work ? t : kPNoTile;
    };

    grid_dependency_wait();   // the set-up above overlaps the tail of the kernel before this one on the stream
    const unsigned int epoch = scan_launch_tag(p.counters);
    if (tid == 0) announce_and_load(draw());
    worker_sync(w);
    uint4 cur = make_uint4(s_next[0], s_next[1], s_next[2], s_next[3]);
    uint32_t tile_phase = 0;          // bar_tma and bar_small complete once per tile, bar_g twice

    while (cur.x != kPNoTile) {
        const int c = (int)cur.x, chain = (int)cur.y, b = (int)cur.z, h = (int)(cur.w & 0x3fffffffu), x = (int)(cur.w >> 30);
        const unsigned int tile = (unsigned)c * (unsigned)p.n_chains + (unsigned)chain;
        uint2* agg_rec = p.agg_rec[x];
        uint2* prefix_rec = p.prefix_rec[x];
        unsigned int t_next = kPNoTile;
        if (tid == 0) t_next = draw();                       // the answer is needed only when this tile's products are done
        const long long cnt0 = p.count_in ? p.count_in[b] : 0ll;
        const int valid = min(kGT, p.S - c * kGT);           // tokens in this tile
        if (EMA && valid != w_valid) {   // a shorter (last) tile, or the first full one after it: other weights in the aggregate
            write_agg_weights(valid);
            w_valid = valid;
            fence_proxy_async();
            worker_sync(w);
        }

        wait_bar_parked(bar_tma, tile_phase, abort_flag, p.wait_cycles, p.status, 200);

        // ---- X^T 1 (columns 64-79) and columns 0-63 of G, issued together ------------------------------------
        if (tid == 0) {
            tc_fence_after();
            mma_burst<kPBlock, true>(k8, tm_s, x_lo | dlo_mn, dhi, x_lo + (kHalf >> 4) | dlo_k, dhi, kIdescAgg);   // 16 tokens per step
            mma_commit(bar_small);
            mma_burst<kPBlock, false>(k8, tm_g, x_lo | dlo_k, dhi, x_lo | dlo_k, dhi, kIdescG64);               // 16 dims per step
            mma_commit(bar_g);
        }
        // ---- look-back requests go out under the products (thread = dim) -------------------------------------------
        const int a0 = c > 0 ? ((c - 1) / kGramAnchorEvery) * kGramAnchorEvery : 0;
        const uint2* prec = prefix_rec + ((size_t)(a0 / kGramAnchorEvery) * p.n_chains + chain) * kHeadDim + tid;
        const uint2* arec = agg_rec + ((size_t)a0 * p.n_chains + chain) * kHeadDim + tid;    // chunk a0 + u: u n_chains records on
        const size_t astride = (size_t)p.n_chains * kHeadDim;
        uint2 pfirst = make_uint2(0, 0), afirst[kPLookBack + 1];
        if (c > 0) {
            pfirst = ld_packet2(prec);
#pragma unroll
            for (int u = 0; u <= kPLookBack; ++u)
                if (a0 + u < c) afirst[u] = ld_packet2(arec + u * astride);
        }

        wait_bar_parked(bar_small, tile_phase, abort_flag, p.wait_cycles, p.status, 201);
        tile_phase ^= 1;
        tc_fence_after();
        float agg;
        {
            uint32_t r0[8];
            tmem_ld8(tm_s + lane_off, r0);
            tmem_wait_ld();
            agg = an.agg_of(r0);
        }
        if (c + 1 < p.n_chunks) st_packet2(agg_rec + (size_t)tile * kHeadDim + tid, agg, epoch);

        // ---- carry: prefix record of chunk a0 + aggregates of chunks a0 .. c-1, in ascending order ---------------------
        float carry = 0.f;
        if (c == 0) {
            if (p.sum_in[x]) carry = p.sum_in[x][(size_t)chain * kHeadDim + tid];
        } else {
            float A = 0.f;
#pragma unroll
            for (int u = 0; u <= kPLookBack; ++u)
                if (a0 + u < c) A = an.look_back(A, wait_packet2(arec + u * astride, afirst[u], epoch, p.max_polls, p.status, tile));
            carry = an.carry_of(wait_packet2(prec, pfirst, epoch, p.max_polls, p.status, tile), A, c - a0);
        }
        if (c % kGramAnchorEvery == 0 && c + 1 < p.n_chunks)
            st_packet2(prefix_rec + ((size_t)(c / kGramAnchorEvery) * p.n_chains + chain) * kHeadDim + tid, carry, epoch);
        if (c + 1 == p.n_chunks && p.sum_out[x]) p.sum_out[x][(size_t)chain * kHeadDim + tid] = an.sum_after(carry, agg, valid);
        {   // the carry as c1 + c2 + c3 (bf16 each) into rows 0-2 of the small operand
            float cr = carry;
#pragma unroll
            for (int n = 0; n < 3; ++n) {
                const unsigned short hb = bf16_bits(cr);
                *reinterpret_cast<unsigned short*>(my + pbt_off(n, tid)) = hb;
                cr -= __uint_as_float((uint32_t)hb << 16);
            }
        }
        float c2 = warp_sum(carry * carry);            // ||C||^2 (worker-wide sum over dims)
        if (lane == 0) red[warp * 2] = c2;

        // thread i adds row i of a 64-column half of G left of the diagonal
        float r_acc = 0.f, r_part = 0.f, g_diag = 0.f;
        auto add_half = [&](int hh) {
#pragma unroll
            for (int lc = 0; lc < 2; ++lc) {
                const int cb = 2 * hh + lc;               // 32-column block of G (warp-uniform comparisons)
                if (cb > warp) continue;
                uint32_t g[32];
                tmem_ld32(tm_g + lane_off + lc * 32, g);
                tmem_wait_ld();
                if (cb < warp) an.full_block(g, r_acc);
                else an.diag_block(g, lane, r_part, g_diag);
            }
        };
        wait_bar_parked(bar_g, 0, abort_flag, p.wait_cycles, p.status, 202);
        tc_fence_after();
        add_half(0);
        fence_proxy_async();
        tc_fence_before();
        worker_sync(w);
        c2 = (red[0] + red[2]) + (red[4] + red[6]);
        // ---- columns 64-127 of G and u = X [c1 c2 c3 ..]^T as one product of 80 columns ------------------------------------
        if (tid == 0) {
            tc_fence_after();
            mma_burst<kPBlock, false>(k8, tm_g, x_lo | dlo_k, dhi, x_lo + (64 * 128 >> 4) | dlo_k, dhi, kIdescG80);
            mma_commit(bar_g);
        }
        wait_bar_parked(bar_g, 1, abort_flag, p.wait_cycles, p.status, 203);
        tc_fence_after();
        // every product that reads this tile has completed: the next one may land on it
        if (tid == 0) announce_and_load(*abort_flag ? kPNoTile : t_next);
        add_half(1);
        float d;
        {
            uint32_t r0[8];
            tmem_ld8(tm_s + lane_off, r0);
            tmem_wait_ld();
            d = an.dot((__uint_as_float(r0[0]) + __uint_as_float(r0[1])) + __uint_as_float(r0[2]), r_acc, r_part);   // <x_i, anchor before token i>
        }

        // ---- ||anchor||^2 before each token by a worker-wide prefix scan of the norm steps, then the cosine -------------
        const float bi = an.norm_step(d, g_diag);
        tc_fence_before();
        float pn = an.norm_before(bi, c2, warp, lane, red + 1, [w] { worker_sync(w); });
        const int t_tok = c * kGT + tid;
        if (t_tok < p.S) {
            if (p.incl) { d += g_diag; pn += bi; }
            const long long cnt = cnt0 + t_tok + (p.incl ? 1 : 0);
            p.sim[x][((size_t)b * p.S + t_tok) * p.H + h] = anchor_cosine<EMA>(d, g_diag, pn, cnt);
        }
        cur = make_uint4(s_next[0], s_next[1], s_next[2], s_next[3]);   // rewritten, like red[], only after the next tile's first worker barrier
    }

    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000ll) { }
        __syncthreads();
    }
    if (threadIdx.x < 32) tmem_dealloc(tmem, kPTmemCols);
    if (threadIdx.x == 0) scan_leave(p.counters, gridDim.x);   // every worker of this CTA has stopped drawing
}

}  // namespace

bool kv_stats_gram_usable(const tf_shape& s, const tf_filter_params& p) {
    (void)p;
    return s.dtype == TF_BF16;      // every anchor mode: running sums (past / inclusive mean) and EMA
}

namespace {
// scratch: the counter words, then per tensor one 1 KiB record (128 packets of 8 bytes) per tile and one per
// kGramAnchorEvery-th chunk of a chain
struct GramLayout { size_t tiles, anchors, agg_offset, prefix_offset, bytes; int n_chains, n_chunks; };
GramLayout gram_layout(const tf_shape& s) {
    GramLayout g{};
    g.n_chains = s.batch * s.n_kv_heads;
    g.n_chunks = (s.seq + kGT - 1) / kGT;
    g.tiles = (size_t)g.n_chains * (size_t)g.n_chunks;
    g.anchors = (size_t)g.n_chains * (size_t)((g.n_chunks + kGramAnchorEvery - 1) / kGramAnchorEvery);
    const size_t rec = kHeadDim * sizeof(uint2);
    g.agg_offset = kScanCounterBytes;
    g.prefix_offset = g.agg_offset + 2 * g.tiles * rec;
    g.bytes = (g.prefix_offset + 2 * g.anchors * rec + 255) / 256 * 256;
    return g;
}
}  // namespace

size_t gram_scratch_bytes(const tf_shape& s) { return gram_layout(s).bytes; }

cudaError_t launch_kv_stats_gram(tf_ctx* ctx, const tf_shape& s, const tf_filter_params& p,
                                 const void* K, const void* V, float* sim_k, float* sim_v,
                                 const tf_carry* carry, ScanScratch* ws, cudaStream_t st) {
    const GramLayout gl = gram_layout(s);
    const size_t tiles = gl.tiles;
    if (tiles == 0) return cudaSuccess;
    if (2 * tiles > 0x7fffffffu) return cudaErrorInvalidValue;
    if (ws->capacity < gl.bytes) return cudaErrorInvalidValue;
    CUtensorMap mk, mv;
    if (!make_bshd_map(&mk, K, s.k_stride, s.batch, s.seq, s.n_kv_heads, 2, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 64, kGT,
                       CU_TENSOR_MAP_SWIZZLE_128B) ||
        !make_bshd_map(&mv, V, s.v_stride, s.batch, s.seq, s.n_kv_heads, 2, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 64, kGT,
                       CU_TENSOR_MAP_SWIZZLE_128B))
        return cudaErrorNotSupported;
    // (the low bit of the layout key distinguishes this record layout from the plain kernel's, which may share the scratch)
    const size_t key = gl.bytes | 1;
    if (ws->needs_clear || ws->bytes != key) {
        cudaError_t e = cudaMemsetAsync(ws->ptr, 0, gl.bytes, st);
        if (e != cudaSuccess) return e;
        ws->needs_clear = false;
        ws->bytes = key;
    }

    static bool attr_set_dev[kDeviceFlagSlots] = {};      // function attributes are per device
    bool& attr_set = attr_set_dev[ctx->device >= 0 && ctx->device < kDeviceFlagSlots ? ctx->device : 0];
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(kv_stats_gram1_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kT1Smem);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(kv_stats_gram1_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kT1Smem);
        if (e != cudaSuccess) return e;
        attr_set = true;
    }
    Gram1Params gp{};
    gp.S = s.seq; gp.H = s.n_kv_heads; gp.n_chains = gl.n_chains; gp.n_chunks = gl.n_chunks;
    gp.incl = (p.anchor_mode == TF_ANCHOR_INCL_MEAN);
    const bool ema = (p.anchor_mode == TF_ANCHOR_EMA);
    gp.gamma = ema ? p.gamma : 1.f;
    if (carry) {
        gp.sum_in[0] = carry->sum_k_in; gp.sum_in[1] = carry->sum_v_in;
        gp.count_in = reinterpret_cast<const long long*>(carry->count_in);
        gp.sum_out[0] = carry->sum_k_out; gp.sum_out[1] = carry->sum_v_out;
    }
    gp.sim[0] = sim_k; gp.sim[1] = sim_v;
    char* base = static_cast<char*>(ws->ptr);
    const size_t rec = kHeadDim * sizeof(uint2);
    for (int x = 0; x < 2; ++x) {
        gp.agg_rec[x] = reinterpret_cast<uint2*>(base + gl.agg_offset + x * tiles * rec);
        gp.prefix_rec[x] = reinterpret_cast<uint2*>(base + gl.prefix_offset + x * gl.anchors * rec);
    }
    gp.status = ctx->dev_status;
    gp.max_polls = ctx_max_polls(ctx);
    gp.wait_cycles = ctx_wait_cycles(ctx);
    gp.counters = reinterpret_cast<unsigned int*>(base);
    gp.n_work = (unsigned int)(2 * tiles);
    int sms = 148;
    { int dev = 0; if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev); }
    // the persistent form pays its set-up once per SM and wins once every worker sees several tiles (measured
    // cross-over between 2.3 and 11.5 tiles per worker); below that the one-tile-per-CTA form starts sooner
    const bool persistent = ctx->scan_path == 3 || (ctx->scan_path == 0 && 2 * tiles >= (size_t)4 * sms * kPWorkers);
    cudaError_t e;
    if (persistent) {
        static bool attr_set_p_dev[kDeviceFlagSlots] = {};
        bool& attr_set_p = attr_set_p_dev[ctx->device >= 0 && ctx->device < kDeviceFlagSlots ? ctx->device : 0];
        if (!attr_set_p) {
            e = cudaFuncSetAttribute(kv_stats_gram_persistent_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kPSmem);
            if (e == cudaSuccess) e = cudaFuncSetAttribute(kv_stats_gram_persistent_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kPSmem);
            if (e != cudaSuccess) return e;
            attr_set_p = true;
        }
        const unsigned int grid = std::min<unsigned int>((unsigned int)sms, (gp.n_work + kPWorkers - 1) / kPWorkers);
        GramPParams pp{};
        pp.g = gp;
        e = ema ? launch_dependent(kv_stats_gram_persistent_kernel<true>, dim3(grid), dim3(kPThreads), kPSmem, st, pp, mk, mv)
                : launch_dependent(kv_stats_gram_persistent_kernel<false>, dim3(grid), dim3(kPThreads), kPSmem, st, pp, mk, mv);
        ctx->last_scan_kernel = TF_KERNEL_SCAN_GRAM_PERSISTENT;
    } else {
        e = ema ? launch_dependent(kv_stats_gram1_kernel<true>, dim3(gp.n_work), dim3(128), kT1Smem, st, gp, mk, mv)
                : launch_dependent(kv_stats_gram1_kernel<false>, dim3(gp.n_work), dim3(128), kT1Smem, st, gp, mk, mv);
        ctx->last_scan_kernel = TF_KERNEL_SCAN_GRAM_TILE;
    }
    ctx->launches += 1;
    if (e != cudaSuccess) ws->needs_clear = true;   // whatever the launch left behind is cleared before the next one
    return e;
}

}  // namespace tf
