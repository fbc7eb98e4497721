// Step a5 on the 5th-generation tensor cores: bf16 causal (optionally windowed) attention for
// retained tokens only, head_dim 128.
//
// One CTA owns 128 consecutive entries of a sequence's retained list for one query head.  The
// query rows are gathered (they are scattered in the sequence) into shared memory in the
// 128-byte-swizzled K-major operand layout; K and V tiles of 128 keys are fetched by TMA through
// tensor maps over the caller's strided K/V and consumed in place by tcgen05.mma:
//     S = Q K^T   (A = Q, B = K, both K-major)          -> TMEM, two buffers
//     O += P V    (A = P from shared memory, B = V MN-major, i.e. as it lies in memory) -> TMEM
// Thread r owns row r: it reads its S row from TMEM, applies the row's own causal / window
// limits (row r attends keys up to ITS token position, not the tile diagonal), runs the online
// softmax in fp32, rescales its O row in TMEM when the running maximum moved, and writes P as
// bf16.  QK^T of the next tile is issued before the softmax of the current one, so tensor work
// overlaps the exponentials.  The epilogue normalises, converts to bf16 and scatters rows back
// to their token positions; rows of pruned tokens between two retained tokens are zeroed by the
// thread that owns the later one (Section 3.2: skipped tokens' attention output is zero).
//
// Every mbarrier wait is bounded by a cycle budget; on expiry the CTA records TF_ERR_TIMEOUT,
// stops waiting, releases its TMEM and exits.
#include <cuda.h>

#include "tf_common.cuh"

namespace tf {
namespace {

constexpr int kTileM = 128;           // query rows per CTA
constexpr int kTileN = 128;           // keys per tile
constexpr int kHalfBytes = 128 * 128; // one [128 rows][128 B] swizzled block (64 bf16 per row)
constexpr int kTileBytes = 2 * kHalfBytes;
constexpr int kKvStages = 2;
constexpr uint32_t kTmemCols = 512;
constexpr long long kWaitCycles = 400000000ll;   // ~0.2 s at 2 GHz

struct TcParams {
    const __nv_bfloat16* Q; __nv_bfloat16* O;
    Strides3 qs, os;
    int S, Hq, Hkv, window;
    float scale_log2;
    const int32_t* kept_idx; const int32_t* n_kept;
    DevStatus* status;
};

// shared-memory map (dynamic, base aligned to 1024 B)
constexpr int kOffQ = 0;
constexpr int kOffK = kOffQ + kTileBytes;
constexpr int kOffV = kOffK + kKvStages * kTileBytes;
constexpr int kOffP = kOffV + kKvStages * kTileBytes;
constexpr int kOffBar = kOffP + kTileBytes;
constexpr int kSmemBytes = kOffBar + 256 + 1024;   // barriers + alignment slack

// ---- PTX wrappers -------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" :: "r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// bounded wait; after the first expiry in this CTA nobody waits any more
__device__ __forceinline__ void mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          DevStatus* status, unsigned long long where) {
    if (mbar_try_wait(bar, parity)) return;
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity)) {
        if (*abort_flag) return;
        if (clock64() - t0 > kWaitCycles) {
            *abort_flag = 1;
            report_error(status, TF_ERR_TIMEOUT, where);
            return;
        }
    }
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar,
                                            int c0, int c1, int c2, int c3) {
    asm volatile("cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
                 :: "r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" :: "r"(dst_smem), "r"(cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t addr, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(addr), "r"(cols) : "memory");
}
// D[tmem] (+)= A[smem desc] * B[smem desc]
__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
                 :: "r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void mma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" :: "r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t* r) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                 "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                   "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                   "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                 : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t* r) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
                 "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
                 :: "r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
                    "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
                    "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
                    "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
                 : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    uint32_t d;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}

// Shared-memory operand descriptors (sm_100 format: version 1 at bit 46, swizzle mode at 61-63).
// All operand blocks here are [rows][128 B] with the 128-byte swizzle; groups of 8 rows are 1024 B apart.
//   K-major operand (Q, K, P): rows are M/N, the 128 B hold 64 consecutive K elements.
//   MN-major operand (V):      rows are K (keys), the 128 B hold 64 consecutive N elements (dims);
//                              the next 64 dims start one 16 KiB block later (leading byte offset).
__device__ __forceinline__ uint64_t desc_kmajor(uint32_t addr) {
    return (uint64_t)((addr & 0x3ffffu) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) |
           ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
__device__ __forceinline__ uint64_t desc_mnmajor(uint32_t addr) {
    return (uint64_t)((addr & 0x3ffffu) >> 4) | ((uint64_t)(kHalfBytes >> 4) << 16) | ((uint64_t)(1024 >> 4) << 32) |
           ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
// instruction descriptor: D fp32, A/B bf16, M=128, N=128; bit 16 set = B is MN-major
constexpr uint32_t kIdescQK = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((128u >> 4) << 24);
constexpr uint32_t kIdescPV = kIdescQK | (1u << 16);

// byte offset of 16-byte chunk cc (0..15) of row r inside a two-block [128][64]+[128][64] operand
__device__ __forceinline__ uint32_t swz(int r, int cc) {
    return (uint32_t)((cc >> 3) * kHalfBytes + r * 128 + (((cc & 7) ^ (r & 7)) << 4));
}

__global__ void __launch_bounds__(kTileM, 1)
attention_tc_kernel(const TcParams p, const __grid_constant__ CUtensorMap mapK, const __grid_constant__ CUtensorMap mapV) {
    extern __shared__ uint8_t smem_raw[];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int tile = gridDim.x - 1 - blockIdx.x;   // heaviest tiles first
    const int qh = blockIdx.y, b = blockIdx.z;
    const int nk = p.n_kept[b];
    const int slot0 = tile * kTileM;
    if (slot0 >= max(nk, 1)) return;

    const int32_t* kept = p.kept_idx + (size_t)b * p.S;
    __nv_bfloat16* Ob = p.O + (long long)b * p.os.b + (long long)qh * p.os.h;
    const uint4 zero4 = make_uint4(0, 0, 0, 0);
    if (nk == 0) {   // nothing retained: the whole head is zero
        for (int i = tid; i < p.S * 16; i += kTileM)
            *reinterpret_cast<uint4*>(Ob + (long long)(i >> 4) * p.os.t + (i & 15) * 8) = zero4;
        return;
    }

    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const uint32_t sbase = smem_u32(smem);
    const uint32_t bar_k = sbase + kOffBar, bar_v = bar_k + 16, bar_s = bar_v + 16, bar_o = bar_s + 16;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + kOffBar + 64);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + kOffBar + 72);

    // ---- this thread's row ------------------------------------------------------------------------
    const int slot = slot0 + tid;
    const bool valid = slot < nk;
    const int t_row = valid ? kept[slot] : -1;
    const int hi = t_row;
    const int lo = (valid && p.window > 0) ? max(0, t_row - p.window + 1) : 0;
    const int t_first = kept[slot0];
    const int t_last = kept[min(slot0 + kTileM, nk) - 1];
    const int j_begin = ((p.window > 0 ? max(0, t_first - p.window + 1) : 0) / kTileN) * kTileN;
    const int n_tiles = (t_last - j_begin) / kTileN + 1;
    const int kh = qh / (p.Hq / p.Hkv);

    if (tid == 0) {
        for (int i = 0; i < 2; ++i) { mbar_init(bar_k + 8 * i, 1); mbar_init(bar_v + 8 * i, 1); mbar_init(bar_s + 8 * i, 1); }
        mbar_init(bar_o, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    if (warp == 0) tmem_alloc(smem_u32(tmem_slot), kTmemCols);

    // ---- zero the rows of pruned tokens that precede this row (and follow the last retained one) ---
    if (valid) {
        const int prev = slot == 0 ? -1 : kept[slot - 1];
        for (int t = prev + 1; t < t_row; ++t)
            for (int c = 0; c < 16; ++c) *reinterpret_cast<uint4*>(Ob + (long long)t * p.os.t + c * 8) = zero4;
        if (slot == nk - 1)
            for (int t = t_row + 1; t < p.S; ++t)
                for (int c = 0; c < 16; ++c) *reinterpret_cast<uint4*>(Ob + (long long)t * p.os.t + c * 8) = zero4;
    }

    // ---- gather Q rows into the swizzled K-major operand layout ---------------------------------
    {
        const __nv_bfloat16* qrow = p.Q + (long long)b * p.qs.b + (long long)max(t_row, 0) * p.qs.t + (long long)qh * p.qs.h;
#pragma unroll
        for (int cc = 0; cc < 16; ++cc) {
            const uint4 v = valid ? ldg16(qrow + cc * 8) : zero4;
            *reinterpret_cast<uint4*>(smem + kOffQ + swz(tid, cc)) = v;
        }
    }
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    const uint32_t tm_lane = tmem + ((uint32_t)(warp * 32) << 16);   // this warp's 32 TMEM lanes
    const uint32_t tm_o = tm_lane + 256;

    auto load_k = [&](int it) {
        const int st = it % kKvStages;
        mbar_expect_tx(bar_k + 8 * st, kTileBytes);
        tma_load_4d(sbase + kOffK + st * kTileBytes, &mapK, bar_k + 8 * st, 0, kh, j_begin + it * kTileN, b);
        tma_load_4d(sbase + kOffK + st * kTileBytes + kHalfBytes, &mapK, bar_k + 8 * st, 64, kh, j_begin + it * kTileN, b);
    };
    auto load_v = [&](int it) {
        const int st = it % kKvStages;
        mbar_expect_tx(bar_v + 8 * st, kTileBytes);
        tma_load_4d(sbase + kOffV + st * kTileBytes, &mapV, bar_v + 8 * st, 0, kh, j_begin + it * kTileN, b);
        tma_load_4d(sbase + kOffV + st * kTileBytes + kHalfBytes, &mapV, bar_v + 8 * st, 64, kh, j_begin + it * kTileN, b);
    };
    auto issue_qk = [&](int it) {   // S[it % 2] = Q K[it]^T, 8 steps of 16 dims
        const uint32_t kaddr = sbase + kOffK + (it % kKvStages) * kTileBytes;
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
            const uint32_t off = (kk >> 2) * kHalfBytes + (kk & 3) * 32;
            mma_ss(tmem + (it & 1) * 128, desc_kmajor(sbase + kOffQ + off), desc_kmajor(kaddr + off), kIdescQK, kk > 0);
        }
        mma_commit(bar_s + 8 * (it & 1));
    };
    auto issue_pv = [&](int it) {   // O (+)= P V[it], 8 steps of 16 keys
        const uint32_t vaddr = sbase + kOffV + (it % kKvStages) * kTileBytes;
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
            const uint32_t poff = (kk >> 2) * kHalfBytes + (kk & 3) * 32;
            mma_ss(tmem + 256, desc_kmajor(sbase + kOffP + poff), desc_mnmajor(vaddr + kk * 16 * 128), kIdescPV,
                   (it > 0 || kk > 0) ? 1u : 0u);
        }
        mma_commit(bar_o);
    };

    if (tid == 0) {
        load_k(0); load_v(0);
        if (n_tiles > 1) load_k(1);
        mbar_wait(bar_k, 0, abort_flag, p.status, 1);
        tc_fence_after();
        issue_qk(0);
    }
    __syncwarp();

    float m_run = -INFINITY, l_run = 0.f;
    for (int it = 0; it < n_tiles; ++it) {
        const int j0 = j_begin + it * kTileN;
        // ---- S(it) is ready; get QK(it+1) going before the softmax ---------------------------------
        mbar_wait(bar_s + 8 * (it & 1), (it >> 1) & 1, abort_flag, p.status, 2);
        __syncwarp();
        tc_fence_after();
        if (tid == 0 && it + 1 < n_tiles) {
            // K stage of tile it is free now (QK(it) done): fetch K(it+2) into it
            if (it + 2 < n_tiles) load_k(it + 2);
            mbar_wait(bar_k + 8 * ((it + 1) % kKvStages), ((it + 1) / kKvStages) & 1, abort_flag, p.status, 3);
            tc_fence_after();
            issue_qk(it + 1);
        }
        __syncwarp();   // the .sync.aligned TMEM accesses below need the whole warp together
        // ---- softmax of row `tid` over the 128 keys of this tile ----------------------------------
        uint32_t sreg[128];
#pragma unroll
        for (int c = 0; c < 4; ++c) tmem_ld32(tm_lane + (it & 1) * 128 + c * 32, sreg + c * 32);
        tmem_wait_ld();
        const bool full = (j0 >= lo) && (j0 + kTileN - 1 <= hi);
        float mx = -INFINITY;
        if (full) {
#pragma unroll
            for (int c = 0; c < 128; ++c) mx = fmaxf(mx, __uint_as_float(sreg[c]));
        } else {
#pragma unroll
            for (int c = 0; c < 128; ++c) {
                const int j = j0 + c;
                const float s = (j >= lo && j <= hi) ? __uint_as_float(sreg[c]) : -INFINITY;
                sreg[c] = __float_as_uint(s);
                mx = fmaxf(mx, s);
            }
        }
        const float m_new = fmaxf(m_run, mx * p.scale_log2);
        const float m_safe = (m_new == -INFINITY) ? 0.f : m_new;
        const float corr = ex2(m_run - m_safe);
        float psum = 0.f;
        uint32_t pk[64];
#pragma unroll
        for (int c = 0; c < 64; ++c) {
            const float p0 = ex2(fmaf(__uint_as_float(sreg[2 * c]), p.scale_log2, -m_safe));
            const float p1 = ex2(fmaf(__uint_as_float(sreg[2 * c + 1]), p.scale_log2, -m_safe));
            psum += p0 + p1;
            pk[c] = pack_bf16(p0, p1);
        }
        l_run = fmaf(l_run, corr, psum);
        m_run = m_new;

        // ---- PV(it-1) must be complete before O is rescaled and P overwritten ---------------------
        if (it > 0) {
            mbar_wait(bar_o, (it - 1) & 1, abort_flag, p.status, 4);
            tc_fence_after();
            if (tid == 0 && it + 1 < n_tiles) load_v(it + 1);   // V stage of tile it-1 is free now
            __syncwarp();
            if (__any_sync(0xffffffffu, corr != 1.f)) {
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    uint32_t o[32];
                    tmem_ld32(tm_o + c * 32, o);
                    tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * corr);
                    tmem_st32(tm_o + c * 32, o);
                }
                tmem_wait_st();
            }
        } else if (tid == 0 && n_tiles > 1) {
            load_v(1);
        }
#pragma unroll
        for (int cc = 0; cc < 16; ++cc)
            *reinterpret_cast<uint4*>(smem + kOffP + swz(tid, cc)) = make_uint4(pk[4 * cc], pk[4 * cc + 1], pk[4 * cc + 2], pk[4 * cc + 3]);
        fence_proxy_async();
        tc_fence_before();
        __syncthreads();
        if (tid == 0) {
            tc_fence_after();
            mbar_wait(bar_v + 8 * (it % kKvStages), (it / kKvStages) & 1, abort_flag, p.status, 5);
            tc_fence_after();
            issue_pv(it);
        }
    }

    // ---- epilogue: O / l -> bf16 -> the row's token position ------------------------------------
    mbar_wait(bar_o, (n_tiles - 1) & 1, abort_flag, p.status, 6);
    __syncwarp();
    tc_fence_after();
    {
        const float inv = 1.f / l_run;
        __nv_bfloat16* orow = Ob + (long long)max(t_row, 0) * p.os.t;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            uint32_t o[32];
            tmem_ld32(tm_o + c * 32, o);
            tmem_wait_ld();
            if (valid) {
#pragma unroll
                for (int v = 0; v < 4; ++v) {
                    uint4 w;
                    w.x = pack_bf16(__uint_as_float(o[8 * v + 0]) * inv, __uint_as_float(o[8 * v + 1]) * inv);
                    w.y = pack_bf16(__uint_as_float(o[8 * v + 2]) * inv, __uint_as_float(o[8 * v + 3]) * inv);
                    w.z = pack_bf16(__uint_as_float(o[8 * v + 4]) * inv, __uint_as_float(o[8 * v + 5]) * inv);
                    w.w = pack_bf16(__uint_as_float(o[8 * v + 6]) * inv, __uint_as_float(o[8 * v + 7]) * inv);
                    *reinterpret_cast<uint4*>(orow + c * 32 + v * 8) = w;
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {   // a wait gave up: give copies and MMAs still in flight time to land before leaving
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000ll) { }
        __syncthreads();
    }
    if (warp == 0) tmem_dealloc(tmem, kTmemCols);
}

// ---- host side: tensor maps over the caller's K / V ----------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* sym = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(sym);
    }
    return fn;
}

bool make_kv_map(CUtensorMap* map, const void* base, const int64_t st[3], int B, int S, int H) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    // dims (fastest first): head_dim, head, token, batch
    const cuuint64_t dims[4] = {(cuuint64_t)kHeadDim, (cuuint64_t)H, (cuuint64_t)S, (cuuint64_t)B};
    const cuuint64_t strides[3] = {(cuuint64_t)st[2] * 2, (cuuint64_t)st[1] * 2,
                                   (cuuint64_t)(st[0] > 0 ? st[0] : (int64_t)S * st[1]) * 2};
    const cuuint32_t box[4] = {64, 1, (cuuint32_t)kTileN, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

cudaError_t launch_attention_tc(tf_ctx* ctx, const tf_shape& s, const tf_filter_params& p,
                                const void* Q, const void* K, const void* V,
                                const int32_t* kept_idx, const int32_t* n_kept, void* O,
                                cudaStream_t st) {
    (void)p;
    if (s.dtype != TF_BF16 || s.head_dim != kHeadDim) return cudaErrorNotSupported;
    if (s.batch == 0 || s.seq == 0) return cudaSuccess;
    CUtensorMap mapK, mapV;
    if (!make_kv_map(&mapK, K, s.k_stride, s.batch, s.seq, s.n_kv_heads) ||
        !make_kv_map(&mapV, V, s.v_stride, s.batch, s.seq, s.n_kv_heads))
        return cudaErrorNotSupported;
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(attention_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
        if (e != cudaSuccess) return e;
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
    const dim3 grid((unsigned)((s.seq + kTileM - 1) / kTileM), (unsigned)s.n_q_heads, (unsigned)s.batch);
    attention_tc_kernel<<<grid, kTileM, kSmemBytes, st>>>(tp, mapK, mapV);
    ctx->launches += 1;
    return cudaGetLastError();
}

}  // namespace tf
