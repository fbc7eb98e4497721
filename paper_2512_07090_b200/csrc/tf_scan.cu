// Steps a1-a3 of the Token Filtering layer: anchors, per-head cosine similarity, fused score.
//
// kv_stats_kernel: single pass over K and V.  The running sum of past tokens (the anchor up to
// a scale factor, Alg. 1 "AnchorK <- mean(K)") is a prefix sum along the sequence per (batch,
// kv head, dim).  A CTA owns one chunk of tokens of one head, keeps that chunk in registers,
// and resolves the sum of everything before its chunk with a chained scan over per-chunk
// records in global memory:
//   - every chunk publishes its aggregate; every kAnchorEvery-th chunk also publishes its
//     exclusive prefix P;
//   - chunk c takes P of the nearest earlier anchor chunk a and adds the aggregates a..c-1 in
//     ascending order.  The association is fixed, so results do not depend on timing.
// A record is 128 16-byte packets {k value, v value, tag, 0}; a packet is valid when its tag is
// this launch's tag (derived from a launch counter in the scratch itself), so value and validity arrive in one load and nothing is cleared between
// launches.  Tiles are handed out by an atomic ticket, chunk index slowest, so every record a
// running tile waits for belongs to a tile that has itself started: the waits cannot deadlock,
// and every wait is bounded anyway (on expiry the kernel records TF_ERR_TIMEOUT and goes on).
// The last CTA to have drawn its ticket sets the counter back to zero for the next launch.
//
// Inside the CTA, 8 lanes share a token row (16 dims each, two 16-byte loads for bf16) and 16
// such groups take consecutive runs of tokens; the groups' local sums are scanned through
// shared memory.  Bytes moved: K and V once, 8 bytes of similarity per (token, head) out,
// 2 KiB of record per 32 KiB tile.
#include "tf_common.cuh"

namespace tf {

constexpr int kScanThreads = 128;
constexpr int kGroupLanes = 8;
constexpr int kGroups = kScanThreads / kGroupLanes;  // 16 token runs per CTA
constexpr int kDimsPerLane = kHeadDim / kGroupLanes;  // 16

template <typename T> struct ScanCfg;
template <> struct ScanCfg<float> { static constexpr int kTokPerGroup = 2; };
template <> struct ScanCfg<__nv_bfloat16> { static constexpr int kTokPerGroup = 4; };

constexpr int kAnchorEvery = 8;   // every 8th chunk of a chain publishes its exclusive prefix
constexpr int kPollBatch = 4;     // record packets requested together while looking back

struct ScanParams {
    const void* K; const void* V;
    Strides3 ks, vs;
    int S, H, n_chains, n_chunks;
    int incl;                 // 1: anchor includes the current token
    float decay, weight;      // anchor <- decay*anchor + weight*x   (1,1 for running sums)
    const float* sum_k_in; const float* sum_v_in; const long long* count_in;
    float* sum_k_out; float* sum_v_out;
    float* sim_k; float* sim_v;
    unsigned int* counters;   // {ticket, finished, launches}: see ScanScratch
    unsigned int n_tiles;
    uint4* agg_rec;      // [tile][128] packets, tile = chunk * n_chains + chain
    uint4* prefix_rec;   // [(chunk / kAnchorEvery) * n_chains + chain][128] packets
    DevStatus* status;
    int max_polls;
};

// 16-byte packets go straight to / come straight from L2 as single transactions
__device__ __forceinline__ uint4 ld_packet(const uint4* p) {
    uint4 r;
    asm volatile("ld.volatile.global.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p) : "memory");
    return r;
}
__device__ __forceinline__ void st_packet(uint4* p, float k, float v, unsigned int tag) {
    asm volatile("st.volatile.global.v4.u32 [%0], {%1,%2,%3,%4};"
                 :: "l"(p), "r"(__float_as_uint(k)), "r"(__float_as_uint(v)), "r"(tag), "r"(0u) : "memory");
}
// wait (bounded) until the packet at p carries this launch's tag
__device__ __forceinline__ uint4 wait_packet(const uint4* p, uint4 first, unsigned int epoch, int max_polls,
                                             DevStatus* status, unsigned long long where) {
    uint4 r = first;
    int polls = 0;
    while (r.z != epoch) {
        if (++polls > max_polls) {
            report_error(status, TF_ERR_TIMEOUT, where);
            r = make_uint4(0u, 0u, epoch, 0u);
            break;
        }
        __nanosleep(32);
        r = ld_packet(p);
    }
    return r;
}

// dim owned by (vector j, lane l, element e): vectors of one row are interleaved across the
// 8 lanes so that each 16-byte load instruction of a group covers 128 contiguous bytes.
template <typename T> __device__ __forceinline__ int dim_of(int j, int l, int e) {
    return j * (kGroupLanes * Elem<T>::kPerVec) + l * Elem<T>::kPerVec + e;
}

template <typename T, bool EMA>
__global__ void __launch_bounds__(kScanThreads, 4) kv_stats_kernel(const ScanParams p) {
    constexpr int TPG = ScanCfg<T>::kTokPerGroup;
    constexpr int CH = kGroups * TPG;
    constexpr int NV = Elem<T>::kVecPerLane, EPV = Elem<T>::kPerVec;

    __shared__ __align__(16) float sub[2][kGroups][kHeadDim];
    __shared__ unsigned int s_ticket, s_tag;

    const int tid = threadIdx.x, g = tid >> 3, l = tid & 7;
    if (tid == 0) {
        s_tag = scan_launch_tag(p.counters);
        s_ticket = scan_draw_ticket(p.counters);
        scan_leave(p.counters, gridDim.x);        // one ticket per CTA: this CTA draws no more
    }
    __syncthreads();
    const unsigned int tile = s_ticket, epoch = s_tag;
    if (tile >= p.n_tiles) return;                // cannot happen while the counters are intact; never index records with it
    const int c = (int)(tile / (unsigned)p.n_chains), chain = (int)(tile % (unsigned)p.n_chains);
    const int b = chain / p.H, h = chain % p.H;
    const int t0 = c * CH + g * TPG;

    // ---- load this group's token rows (registers hold the packed input until the end) ----------
    uint4 kr[TPG][NV], vr[TPG][NV];
    {
        const T* Kb = reinterpret_cast<const T*>(p.K) + (long long)b * p.ks.b + (long long)h * p.ks.h;
        const T* Vb = reinterpret_cast<const T*>(p.V) + (long long)b * p.vs.b + (long long)h * p.vs.h;
#pragma unroll
        for (int i = 0; i < TPG; ++i) {
            const int t = t0 + i;
            if (t < p.S) {
                const T* kp = Kb + (long long)t * p.ks.t + l * EPV;
                const T* vp = Vb + (long long)t * p.vs.t + l * EPV;
#pragma unroll
                for (int j = 0; j < NV; ++j) {
                    kr[i][j] = ldg16_stream(kp + j * (kGroupLanes * EPV));
                    vr[i][j] = ldg16_stream(vp + j * (kGroupLanes * EPV));
                }
            } else {
#pragma unroll
                for (int j = 0; j < NV; ++j) { kr[i][j] = make_uint4(0, 0, 0, 0); vr[i][j] = make_uint4(0, 0, 0, 0); }
            }
        }
    }
    const float a = p.decay, w = p.weight;

    // ---- phase 1: this group's local anchor contribution, started from zero ------------------------
    {
        float sk[kDimsPerLane], sv[kDimsPerLane];
#pragma unroll
        for (int i = 0; i < kDimsPerLane; ++i) { sk[i] = 0.f; sv[i] = 0.f; }
#pragma unroll
        for (int i = 0; i < TPG; ++i) {
            if (t0 + i < p.S) {
                float fk[kDimsPerLane], fv[kDimsPerLane];
#pragma unroll
                for (int j = 0; j < NV; ++j) { Elem<T>::unpack(kr[i][j], fk + j * EPV); Elem<T>::unpack(vr[i][j], fv + j * EPV); }
#pragma unroll
                for (int e = 0; e < kDimsPerLane; ++e) {
                    if (EMA) { sk[e] = fmaf(a, sk[e], w * fk[e]); sv[e] = fmaf(a, sv[e], w * fv[e]); }
                    else     { sk[e] += fk[e]; sv[e] += fv[e]; }
                }
            }
        }
#pragma unroll
        for (int j = 0; j < NV; ++j)
#pragma unroll
            for (int e = 0; e < EPV; ++e) {
                sub[0][g][dim_of<T>(j, l, e)] = sk[j * EPV + e];
                sub[1][g][dim_of<T>(j, l, e)] = sv[j * EPV + e];
            }
    }
    __syncthreads();

    // ---- chunk aggregate of column `tid` (both tensors), then the carry from earlier chunks -------
    // apow[n] = decay^n for a run of n valid tokens
    float apow[TPG + 1];
    apow[0] = 1.f;
#pragma unroll
    for (int n = 1; n <= TPG; ++n) apow[n] = EMA ? apow[n - 1] * a : 1.f;
    const int chunk_valid = min(CH, p.S - c * CH);        // >= 1
    float agg_k = 0.f, agg_v = 0.f, a_chunk = 1.f;
#pragma unroll
    for (int gg = 0; gg < kGroups; ++gg) {
        const int len = max(0, min(TPG, chunk_valid - gg * TPG));
        const float f = apow[len];
        agg_k = EMA ? fmaf(f, agg_k, sub[0][gg][tid]) : agg_k + sub[0][gg][tid];
        agg_v = EMA ? fmaf(f, agg_v, sub[1][gg][tid]) : agg_v + sub[1][gg][tid];
        a_chunk *= f;
    }

    // every chunk but the last of its chain publishes its aggregate
    if (c + 1 < p.n_chunks) st_packet(p.agg_rec + (size_t)tile * kHeadDim + tid, agg_k, agg_v, epoch);

    float carry_k = 0.f, carry_v = 0.f;
    if (c == 0) {
        if (p.sum_k_in) carry_k = p.sum_k_in[(size_t)chain * kHeadDim + tid];
        if (p.sum_v_in) carry_v = p.sum_v_in[(size_t)chain * kHeadDim + tid];
    } else {
        const int a0 = ((c - 1) / kAnchorEvery) * kAnchorEvery;   // nearest earlier anchor chunk
        float a_full = 1.f;                                        // decay of one full chunk
        if (EMA) { for (int n = 0; n < CH; ++n) a_full *= a; }
        const uint4* prec = p.prefix_rec + ((size_t)(a0 / kAnchorEvery) * p.n_chains + chain) * kHeadDim + tid;
        uint4 pfirst = ld_packet(prec);
        float Ak = 0.f, Av = 0.f, decay_to_here = 1.f;
        for (int j0 = a0; j0 < c; j0 += kPollBatch) {
            uint4 r[kPollBatch];
#pragma unroll
            for (int u = 0; u < kPollBatch; ++u)
                if (j0 + u < c) r[u] = ld_packet(p.agg_rec + ((size_t)(j0 + u) * p.n_chains + chain) * kHeadDim + tid);
#pragma unroll
            for (int u = 0; u < kPollBatch; ++u) {
                if (j0 + u < c) {
                    r[u] = wait_packet(p.agg_rec + ((size_t)(j0 + u) * p.n_chains + chain) * kHeadDim + tid, r[u],
                                       epoch, p.max_polls, p.status, tile);
                    Ak = EMA ? fmaf(a_full, Ak, __uint_as_float(r[u].x)) : Ak + __uint_as_float(r[u].x);
                    Av = EMA ? fmaf(a_full, Av, __uint_as_float(r[u].y)) : Av + __uint_as_float(r[u].y);
                    decay_to_here *= a_full;
                }
            }
        }
        pfirst = wait_packet(prec, pfirst, epoch, p.max_polls, p.status, tile);
        carry_k = EMA ? fmaf(decay_to_here, __uint_as_float(pfirst.x), Ak) : __uint_as_float(pfirst.x) + Ak;
        carry_v = EMA ? fmaf(decay_to_here, __uint_as_float(pfirst.y), Av) : __uint_as_float(pfirst.y) + Av;
    }
    if (c % kAnchorEvery == 0 && c + 1 < p.n_chunks)
        st_packet(p.prefix_rec + ((size_t)(c / kAnchorEvery) * p.n_chains + chain) * kHeadDim + tid, carry_k, carry_v, epoch);
    if (c + 1 == p.n_chunks) {
        if (p.sum_k_out) p.sum_k_out[(size_t)chain * kHeadDim + tid] = fmaf(a_chunk, carry_k, agg_k);
        if (p.sum_v_out) p.sum_v_out[(size_t)chain * kHeadDim + tid] = fmaf(a_chunk, carry_v, agg_v);
    }
    // exclusive scan of the groups' contributions, seeded with the carry
    {
        float rk = carry_k, rv = carry_v;
#pragma unroll
        for (int gg = 0; gg < kGroups; ++gg) {
            const int len = max(0, min(TPG, chunk_valid - gg * TPG));
            const float f = apow[len];
            const float tk = sub[0][gg][tid], tv = sub[1][gg][tid];
            sub[0][gg][tid] = rk;
            sub[1][gg][tid] = rv;
            rk = EMA ? fmaf(f, rk, tk) : rk + tk;
            rv = EMA ? fmaf(f, rv, tv) : rv + tv;
        }
    }
    __syncthreads();

    // ---- phase 3: walk the run again with the true anchor ------------------------------------------
    float Pk[kDimsPerLane], Pv[kDimsPerLane];
#pragma unroll
    for (int j = 0; j < NV; ++j)
#pragma unroll
        for (int e = 0; e < EPV; ++e) {
            Pk[j * EPV + e] = sub[0][g][dim_of<T>(j, l, e)];
            Pv[j * EPV + e] = sub[1][g][dim_of<T>(j, l, e)];
        }
    const long long n_before = (p.count_in ? p.count_in[b] : 0ll) + t0;
#pragma unroll
    for (int i = 0; i < TPG; ++i) {
        const int t = t0 + i;
        if (t >= p.S) break;
        float fk[kDimsPerLane], fv[kDimsPerLane];
#pragma unroll
        for (int j = 0; j < NV; ++j) { Elem<T>::unpack(kr[i][j], fk + j * EPV); Elem<T>::unpack(vr[i][j], fv + j * EPV); }
        if (p.incl) {
#pragma unroll
            for (int e = 0; e < kDimsPerLane; ++e) {
                Pk[e] = EMA ? fmaf(a, Pk[e], w * fk[e]) : Pk[e] + fk[e];
                Pv[e] = EMA ? fmaf(a, Pv[e], w * fv[e]) : Pv[e] + fv[e];
            }
        }
        float dk = 0.f, kk = 0.f, pk = 0.f, dv = 0.f, vv = 0.f, pv = 0.f;
#pragma unroll
        for (int e = 0; e < kDimsPerLane; ++e) {
            dk = fmaf(fk[e], Pk[e], dk); kk = fmaf(fk[e], fk[e], kk); pk = fmaf(Pk[e], Pk[e], pk);
            dv = fmaf(fv[e], Pv[e], dv); vv = fmaf(fv[e], fv[e], vv); pv = fmaf(Pv[e], Pv[e], pv);
        }
#pragma unroll
        for (int o = 1; o < kGroupLanes; o <<= 1) {
            dk += __shfl_xor_sync(0xffffffffu, dk, o); kk += __shfl_xor_sync(0xffffffffu, kk, o);
            pk += __shfl_xor_sync(0xffffffffu, pk, o); dv += __shfl_xor_sync(0xffffffffu, dv, o);
            vv += __shfl_xor_sync(0xffffffffu, vv, o); pv += __shfl_xor_sync(0xffffffffu, pv, o);
        }
        const long long n = n_before + i + (p.incl ? 1 : 0);   // tokens the anchor covers
        if (l < 2) {
            const float d = l ? dv : dk, xx = l ? vv : kk, pp = l ? pv : pk;
            float cosv = 0.f;
            if (n > 0) {
                const float s = EMA ? 1.f : 1.f / (float)n;   // anchor = sum * s
                cosv = (d * s) / (fmaxf(sqrtf(xx), kNormEps) * fmaxf(sqrtf(pp) * s, kNormEps));
            }
            float* out = l ? p.sim_v : p.sim_k;
            out[((size_t)b * p.S + t) * p.H + h] = cosv;
        }
        if (!p.incl) {
#pragma unroll
            for (int e = 0; e < kDimsPerLane; ++e) {
                Pk[e] = EMA ? fmaf(a, Pk[e], w * fk[e]) : Pk[e] + fk[e];
                Pv[e] = EMA ? fmaf(a, Pv[e], w * fv[e]) : Pv[e] + fv[e];
            }
        }
    }
}

ScanPlan scan_plan(const tf_shape& s) {
    ScanPlan pl;
    pl.chunk_tokens = kGroups * (s.dtype == TF_BF16 ? ScanCfg<__nv_bfloat16>::kTokPerGroup
                                                   : ScanCfg<float>::kTokPerGroup);
    pl.n_chains = s.batch * s.n_kv_heads;
    pl.n_chunks = (s.seq + pl.chunk_tokens - 1) / pl.chunk_tokens;
    const size_t tiles = (size_t)pl.n_chains * (size_t)pl.n_chunks;
    const size_t anchors = (size_t)pl.n_chains * (size_t)((pl.n_chunks + kAnchorEvery - 1) / kAnchorEvery);
    pl.agg_offset = kScanCounterBytes;                                    // after the counter words
    pl.prefix_offset = pl.agg_offset + tiles * kHeadDim * sizeof(uint4);
    pl.bytes = pl.prefix_offset + anchors * kHeadDim * sizeof(uint4);
    pl.bytes = (pl.bytes + 255) / 256 * 256;
    return pl;
}

cudaError_t launch_kv_stats(tf_ctx* ctx, const tf_shape& s, const tf_filter_params& p,
                            const void* K, const void* V, float* sim_k, float* sim_v,
                            const tf_carry* carry, ScanScratch* ws, cudaStream_t st) {
    if (ctx->scan_path != 1 && kv_stats_gram_usable(s, p)) {
        const cudaError_t e = launch_kv_stats_gram(ctx, s, p, K, V, sim_k, sim_v, carry, ws, st);
        // an explicitly requested kernel is a requirement; the default falls back only when no tensor map can
        // describe the caller's layout
        if (e != cudaErrorNotSupported || ctx->scan_path >= 2) return e;
    }
    if (ctx->scan_path >= 2) return cudaErrorNotSupported;
    const ScanPlan pl = scan_plan(s);
    const size_t tiles = (size_t)pl.n_chains * (size_t)pl.n_chunks;
    if (tiles == 0) return cudaSuccess;
    if (tiles > 0x7fffffffu) return cudaErrorInvalidValue;
    // Tags make stale records harmless, except in memory this library has never written: clear a
    // scratch region once when it is first used (and whenever the 32-bit epoch wraps).
    // The region is also cleared when its extent changes: another shape's layout may have put
    // other data where this shape keeps records.
    if (ws->capacity < pl.bytes) return cudaErrorInvalidValue;
    if (ws->needs_clear || ws->bytes != pl.bytes) {
        cudaError_t e = cudaMemsetAsync(ws->ptr, 0, pl.bytes, st);
        if (e != cudaSuccess) return e;
        ws->needs_clear = false;
        ws->bytes = pl.bytes;
    }

    ScanParams sp{};
    sp.K = K; sp.V = V;
    sp.ks = {s.k_stride[0], s.k_stride[1], s.k_stride[2]};
    sp.vs = {s.v_stride[0], s.v_stride[1], s.v_stride[2]};
    sp.S = s.seq; sp.H = s.n_kv_heads; sp.n_chains = pl.n_chains; sp.n_chunks = pl.n_chunks;
    sp.incl = (p.anchor_mode == TF_ANCHOR_INCL_MEAN);
    const bool ema = (p.anchor_mode == TF_ANCHOR_EMA);
    sp.decay = ema ? p.gamma : 1.f;
    sp.weight = ema ? 1.f - p.gamma : 1.f;
    if (carry) {
        sp.sum_k_in = carry->sum_k_in; sp.sum_v_in = carry->sum_v_in;
        sp.count_in = reinterpret_cast<const long long*>(carry->count_in);
        sp.sum_k_out = carry->sum_k_out; sp.sum_v_out = carry->sum_v_out;
    }
    sp.sim_k = sim_k; sp.sim_v = sim_v;
    char* base = static_cast<char*>(ws->ptr);
    sp.counters = reinterpret_cast<unsigned int*>(base);
    sp.n_tiles = (unsigned int)tiles;
    sp.agg_rec = reinterpret_cast<uint4*>(base + pl.agg_offset);
    sp.prefix_rec = reinterpret_cast<uint4*>(base + pl.prefix_offset);
    sp.status = ctx->dev_status;
    sp.max_polls = ctx_max_polls(ctx);

    const dim3 grid((unsigned)tiles), block(kScanThreads);
    if (s.dtype == TF_BF16) {
        if (ema) kv_stats_kernel<__nv_bfloat16, true><<<grid, block, 0, st>>>(sp);
        else     kv_stats_kernel<__nv_bfloat16, false><<<grid, block, 0, st>>>(sp);
    } else {
        if (ema) kv_stats_kernel<float, true><<<grid, block, 0, st>>>(sp);
        else     kv_stats_kernel<float, false><<<grid, block, 0, st>>>(sp);
    }
    ctx->launches += 1;
    ctx->last_scan_kernel = TF_KERNEL_SCAN_PLAIN;
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) ws->needs_clear = true;   // whatever the launch left behind is cleared before the next one
    return e;
}

// ---------------------------------------------------------------------------------------------------
// Step a3: G lanes per
// token, G = 8, 16 or 32 by head count.  Mean and population variance over heads (two passes over the
// similarities), weight alpha per Eq. 2 (either reading), fused score per Eq. 3.
// ---------------------------------------------------------------------------------------------------
template <int G>
__global__ void __launch_bounds__(256) score_fuse_kernel(const float* __restrict__ sim_k,
                                                         const float* __restrict__ sim_v,
                                                         float* __restrict__ score, long long n_tokens,
                                                         int H, int mode, float eps, DevStatus* status) {
    grid_launch_dependents();   // a short kernel: the selection CTAs may become resident while it runs
    grid_dependency_wait();
    const long long tok = ((long long)blockIdx.x * blockDim.x + threadIdx.x) / G;
    const int lane = threadIdx.x & (G - 1);
    const bool live = tok < n_tokens;               // whole groups are live or not; shuffles below stay inside a group
    const float* ck = sim_k + (live ? tok : 0) * H;
    const float* cv = sim_v + (live ? tok : 0) * H;
    auto group_sum = [](float v) {
#pragma unroll
        for (int o = G / 2; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        return v;
    };
    float sk = 0.f, sv = 0.f;
    for (int h = lane; h < H; h += G) { sk += ck[h]; sv += cv[h]; }
    const float inv = 1.f / (float)H;
    sk = group_sum(sk) * inv;
    sv = group_sum(sv) * inv;
    float vk = 0.f, vv = 0.f;
    for (int h = lane; h < H; h += G) {
        const float a = ck[h] - sk, b = cv[h] - sv;
        vk = fmaf(a, a, vk);
        vv = fmaf(b, b, vv);
    }
    vk = group_sum(vk) * inv;
    vv = group_sum(vv) * inv;
    if (lane == 0 && live) {
        const float s = fuse_score(mode, sk, vk, sv, vv, eps);
        score[tok] = s;
        note_nan_score(status, s, (unsigned long long)tok);
    }
}

cudaError_t launch_score_fuse(tf_ctx* ctx, const tf_shape& s, const tf_filter_params& p,
                              const float* sim_k, const float* sim_v, float* score, cudaStream_t st) {
    const long long n = (long long)s.batch * s.seq;
    if (n == 0) return cudaSuccess;
    const float eps = p.var_eps > 0.f ? p.var_eps : 1e-8f;
    const int G = s.n_kv_heads <= 8 ? 8 : (s.n_kv_heads <= 16 ? 16 : 32);
    const unsigned blocks = (unsigned)((n * G + 255) / 256);
    auto kernel = G == 8 ? score_fuse_kernel<8> : (G == 16 ? score_fuse_kernel<16> : score_fuse_kernel<32>);
    cudaError_t e = launch_dependent(kernel, dim3(blocks), dim3(256), 0, st, sim_k, sim_v, score, n,
                                     s.n_kv_heads, p.fuse_mode, eps, ctx->dev_status);
    ctx->launches += 1;
    return e;
}

}  // namespace tf
