// Steps a1-a3 of the Token Filtering layer: anchors, per-head cosine similarity, fused score.
//
// kv_stats_kernel: single pass over K and V.  The running sum of past tokens (the anchor up to
// a scale factor, Alg. 1 "AnchorK <- mean(K)") is a prefix sum along the sequence per (batch,
// kv head, dim).  A CTA owns one chunk of tokens of one head, keeps that chunk in registers,
// and resolves the sum of everything before its chunk with a chained scan: it publishes its
// chunk aggregate, then looks back over its predecessors' records until it meets one whose
// inclusive prefix is known.  Tiles are handed out by an atomic ticket, chunk index slowest,
// so every predecessor of a running tile has itself started: the look-back cannot deadlock,
// and every wait is bounded anyway (on expiry the kernel records TF_ERR_TIMEOUT and goes on).
//
// Inside the CTA, 8 lanes share a token row (16 dims each, two 16-byte loads for bf16) and 16
// such groups take consecutive runs of tokens; the groups' local sums are scanned through
// shared memory.  Bytes moved: K and V once, 8 bytes of similarity per (token, head) out,
// about 1-2 KiB of scan records per 32 KiB tile.
#include "tf_common.cuh"

namespace tf {

constexpr int kScanThreads = 128;
constexpr int kGroupLanes = 8;
constexpr int kGroups = kScanThreads / kGroupLanes;  // 16 token runs per CTA
constexpr int kDimsPerLane = kHeadDim / kGroupLanes;  // 16

template <typename T> struct ScanCfg;
template <> struct ScanCfg<float> { static constexpr int kTokPerGroup = 2; };
template <> struct ScanCfg<__nv_bfloat16> { static constexpr int kTokPerGroup = 4; };

enum : int { kFlagNone = 0, kFlagAggregate = 1, kFlagPrefix = 2, kFlagTimeout = -1 };

struct ScanParams {
    const void* K; const void* V;
    Strides3 ks, vs;
    int S, H, n_chains, n_chunks;
    int incl;                 // 1: anchor includes the current token
    float decay, weight;      // anchor <- decay*anchor + weight*x   (1,1 for running sums)
    const float* sum_k_in; const float* sum_v_in; const long long* count_in;
    float* sum_k_out; float* sum_v_out;
    float* sim_k; float* sim_v;
    unsigned int* ticket; int* flags; float* records;   // records[tile][agg|prefix][k|v][128]
    DevStatus* status;
    int max_polls;
};

__device__ __forceinline__ int ld_acquire(const int* p) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release(int* p, int v) {
    asm volatile("st.release.gpu.global.s32 [%0], %1;" :: "l"(p), "r"(v) : "memory");
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
    __shared__ unsigned int s_ticket;
    __shared__ int s_flag;

    const int tid = threadIdx.x, g = tid >> 3, l = tid & 7;
    if (tid == 0) s_ticket = atomicAdd(p.ticket, 1u);
    __syncthreads();
    const unsigned int tile = s_ticket;
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

    float* rec = p.records + (size_t)tile * (4 * kHeadDim);   // [agg k, agg v, prefix k, prefix v]
    float carry_k = 0.f, carry_v = 0.f;
    if (c == 0) {
        if (p.sum_k_in) carry_k = p.sum_k_in[(size_t)chain * kHeadDim + tid];
        if (p.sum_v_in) carry_v = p.sum_v_in[(size_t)chain * kHeadDim + tid];
    } else {
        long long pred = (long long)tile - p.n_chains;
        // a full predecessor chunk decays the carry by decay^CH
        float a_full = 1.f;
        if (EMA) { for (int n = 0; n < CH; ++n) a_full *= a; }
        float fac = 1.f;
        bool published = false;
        for (;;) {
            if (tid == 0) {
                int f = ld_acquire(p.flags + pred);
                if (f == kFlagNone && published) {
                    int polls = 0;
                    while ((f = ld_acquire(p.flags + pred)) == kFlagNone) {
                        if (++polls > p.max_polls) { f = kFlagTimeout; break; }
                        __nanosleep(64);
                    }
                }
                s_flag = f;
            }
            __syncthreads();
            const int f = s_flag;
            __syncthreads();
            if (f == kFlagNone) {
                // predecessor not ready yet: let our successors see our aggregate, then wait
                __stcg(rec + tid, agg_k);
                __stcg(rec + kHeadDim + tid, agg_v);
                __threadfence();
                __syncthreads();
                if (tid == 0) st_release(p.flags + tile, kFlagAggregate);
                published = true;
                continue;
            }
            if (f == kFlagTimeout) {
                if (tid == 0) report_error(p.status, TF_ERR_TIMEOUT, tile);
                break;
            }
            const float* prec = p.records + (size_t)pred * (4 * kHeadDim);
            if (f == kFlagPrefix) {
                carry_k = fmaf(fac, __ldcg(prec + 2 * kHeadDim + tid), carry_k);
                carry_v = fmaf(fac, __ldcg(prec + 3 * kHeadDim + tid), carry_v);
                break;
            }
            carry_k = fmaf(fac, __ldcg(prec + tid), carry_k);
            carry_v = fmaf(fac, __ldcg(prec + kHeadDim + tid), carry_v);
            fac *= a_full;
            pred -= p.n_chains;
            if (pred < 0) break;   // cannot happen: chunk 0 only ever publishes a prefix
        }
    }
    {
        const float incl_k = fmaf(a_chunk, carry_k, agg_k), incl_v = fmaf(a_chunk, carry_v, agg_v);
        if (c + 1 < p.n_chunks) {
            __stcg(rec + 2 * kHeadDim + tid, incl_k);
            __stcg(rec + 3 * kHeadDim + tid, incl_v);
            __threadfence();
            __syncthreads();
            if (tid == 0) st_release(p.flags + tile, kFlagPrefix);
        } else {
            if (p.sum_k_out) p.sum_k_out[(size_t)chain * kHeadDim + tid] = incl_k;
            if (p.sum_v_out) p.sum_v_out[(size_t)chain * kHeadDim + tid] = incl_v;
        }
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
    size_t flags = 256 + ((tiles * sizeof(int) + 255) / 256) * 256;   // ticket word + flags
    pl.bytes = flags + tiles * 4 * kHeadDim * sizeof(float);
    pl.bytes = (pl.bytes + 255) / 256 * 256;
    return pl;
}

cudaError_t launch_kv_stats(tf_ctx* ctx, const tf_shape& s, const tf_filter_params& p,
                            const void* K, const void* V, float* sim_k, float* sim_v,
                            const tf_carry* carry, void* scan_scratch, cudaStream_t st) {
    const ScanPlan pl = scan_plan(s);
    const size_t tiles = (size_t)pl.n_chains * (size_t)pl.n_chunks;
    if (tiles == 0) return cudaSuccess;
    const size_t flag_bytes = 256 + ((tiles * sizeof(int) + 255) / 256) * 256;
    cudaError_t e = cudaMemsetAsync(scan_scratch, 0, flag_bytes, st);
    if (e != cudaSuccess) return e;

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
    sp.ticket = reinterpret_cast<unsigned int*>(scan_scratch);
    sp.flags = reinterpret_cast<int*>(reinterpret_cast<char*>(scan_scratch) + 256);
    sp.records = reinterpret_cast<float*>(reinterpret_cast<char*>(scan_scratch) + flag_bytes);
    sp.status = ctx->dev_status;
    sp.max_polls = 1 << 20;   // ~64 ns apart plus an L2 round trip each: of the order of a second

    const dim3 grid((unsigned)tiles), block(kScanThreads);
    if (s.dtype == TF_BF16) {
        if (ema) kv_stats_kernel<__nv_bfloat16, true><<<grid, block, 0, st>>>(sp);
        else     kv_stats_kernel<__nv_bfloat16, false><<<grid, block, 0, st>>>(sp);
    } else {
        if (ema) kv_stats_kernel<float, true><<<grid, block, 0, st>>>(sp);
        else     kv_stats_kernel<float, false><<<grid, block, 0, st>>>(sp);
    }
    ctx->launches += 1;
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------------
// Step a3: one warp per token.  Mean and population variance over heads (two passes over the
// registers), weight alpha per Eq. 2 (either reading), fused score per Eq. 3.
// ---------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) score_fuse_kernel(const float* __restrict__ sim_k,
                                                         const float* __restrict__ sim_v,
                                                         float* __restrict__ score, long long n_tokens,
                                                         int H, int mode, float eps, DevStatus* status) {
    const long long tok = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (tok >= n_tokens) return;
    const float* ck = sim_k + tok * H;
    const float* cv = sim_v + tok * H;
    float sk = 0.f, sv = 0.f;
    for (int h = lane; h < H; h += 32) { sk += ck[h]; sv += cv[h]; }
    const float inv = 1.f / (float)H;
    sk = warp_sum(sk) * inv;
    sv = warp_sum(sv) * inv;
    float vk = 0.f, vv = 0.f;
    for (int h = lane; h < H; h += 32) {
        const float a = ck[h] - sk, b = cv[h] - sv;
        vk = fmaf(a, a, vk);
        vv = fmaf(b, b, vv);
    }
    vk = warp_sum(vk) * inv;
    vv = warp_sum(vv) * inv;
    if (lane == 0) {
        float alpha;
        switch (mode) {
            case TF_FUSE_EQ2_LITERAL: alpha = (vk + eps) / (vk + vv + 2.f * eps); break;
            case TF_FUSE_KEY_ONLY: alpha = 1.f; break;
            case TF_FUSE_VALUE_ONLY: alpha = 0.f; break;
            case TF_FUSE_MEAN: alpha = 0.5f; break;
            default: alpha = (vv + eps) / (vk + vv + 2.f * eps); break;
        }
        float s = alpha * sk + (1.f - alpha) * sv;
        s += 0.f;   // -0 -> +0
        score[tok] = s;
        if (s != s && status) {
            atomicAdd(&status->nan_count, 1ull);
            report_error(status, TF_ERR_NAN_SCORE, (unsigned long long)tok);
        }
    }
}

cudaError_t launch_score_fuse(tf_ctx* ctx, const tf_shape& s, const tf_filter_params& p,
                              const float* sim_k, const float* sim_v, float* score, cudaStream_t st) {
    const long long n = (long long)s.batch * s.seq;
    if (n == 0) return cudaSuccess;
    const float eps = p.var_eps > 0.f ? p.var_eps : 1e-8f;
    const long long threads = n * 32;
    const unsigned blocks = (unsigned)((threads + 255) / 256);
    score_fuse_kernel<<<blocks, 256, 0, st>>>(sim_k, sim_v, score, n, s.n_kv_heads, p.fuse_mode, eps,
                                              ctx->dev_status);
    ctx->launches += 1;
    return cudaGetLastError();
}

}  // namespace tf
