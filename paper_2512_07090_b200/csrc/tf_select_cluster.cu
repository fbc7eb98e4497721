// Steps a3 + a4 in one launch, a thread-block cluster per sequence.
//
// The selection of tf_select.cu runs one CTA per sequence, so a batch of 8 sequences of 16384 tokens keeps 8 of
// the GPU's SMs busy for its whole duration, and the fused scores it reads come from a launch of their own.  Here
// a cluster of 4 or 8 CTAs shares a sequence, CTA r of the cluster owning the contiguous token range
// [r L, (r + 1) L), L = 512 KPT:
//   * step a3 (optional, up to 8 KV heads: a row of similarities is then one or two 16-byte loads and a warp reads
//     a contiguous stretch; with more heads a thread per token reads 32 scattered lines per instruction and step a3
//     stays a launch of its own): every thread computes the fused score of its own tokens from the per-head
//     similarities (mean and population variance over heads, Eq. 2 weight, Eq. 3 score) in exactly the order of
//     additions the 8-lanes-per-token kernel of tf_scan.cu uses, so both give the same bits; the scores are written
//     out (they are an output of the layer step) and stay in registers for step a4;
//   * step a4, RATIO mode: the same 4-pass, 8-bit MSB-first radix select over order-preserving keys as the
//     one-CTA kernel.  Each CTA histograms its own candidates; after a cluster barrier every CTA adds up the
//     cluster's histograms through distributed shared memory and takes the same decision (two histogram buffers
//     alternate, so one cluster barrier per pass is enough); once at most 32 candidates share the prefix they are
//     appended to a list in CTA 0's shared memory and every CTA ranks them there instead of further passes;
//   * ranks in index order (which of the tokens that tie with the P-th key go, and where a retained token lands in
//     kept_idx) are a CTA-local scan plus the totals of the CTAs before it in the cluster, again through
//     distributed shared memory.
// Same results as select_kernel, bit for bit: same keys, same tie rule (equal scores go from the highest index
// down), same outputs.
#include <cooperative_groups.h>
#include <math_constants.h>

#include "tf_common.cuh"

namespace cg = cooperative_groups;

namespace tf {
namespace {

constexpr int kCsThreads = 512;
constexpr int kCsWarps = kCsThreads / 32;

struct ClusterSelectParams {
    const float* sim_k; const float* sim_v;   // [B,S,H]; null: the scores are read from `score`
    float* score;                             // [B,S]: written when sim_k is given, read otherwise
    const uint8_t* eligible;                  // [B,S] or null
    const float* threshold;                   // [B] (threshold mode)
    int S, H, warmup, mode, fuse_mode;
    float eps;
    int vec4;                                 // the similarities can be read as float4 (H a multiple of 4, 16-byte aligned)
    long long p_target;                       // floor(ratio*S), computed on the host in double
    uint8_t* keep_mask; int32_t* kept_idx; int32_t* n_kept; float* theta;
    DevStatus* status;
};

// Step a3 for one token by one thread from the token's similarities in registers (up to 8 KV heads; xk[h], xv[h] are
// read for h < H only), in the order of operations of score_fuse_kernel<8>: "lane" l holds head l (0 + x, as the
// kernel's accumulator starts at zero), the 8 partial values are folded in halves (l with l + 4, then + 2, then + 1).
__device__ __forceinline__ float fuse_token8(const float (&xk)[8], const float (&xv)[8], int H, int mode, float eps) {
    auto fold = [](float (&v)[8]) {
#pragma unroll
        for (int o = 4; o > 0; o >>= 1)
#pragma unroll
            for (int l = 0; l < o; ++l) v[l] = __fadd_rn(v[l], v[l + o]);
        return v[0];
    };
    float pk[8], pv[8];
#pragma unroll
    for (int l = 0; l < 8; ++l) {
        pk[l] = l < H ? __fadd_rn(0.f, xk[l]) : 0.f;
        pv[l] = l < H ? __fadd_rn(0.f, xv[l]) : 0.f;
    }
    const float inv = 1.f / (float)H;
    const float sk = __fmul_rn(fold(pk), inv), sv = __fmul_rn(fold(pv), inv);
#pragma unroll
    for (int l = 0; l < 8; ++l) {
        const float a = __fsub_rn(xk[l], sk), b = __fsub_rn(xv[l], sv);
        pk[l] = l < H ? __fmaf_rn(a, a, 0.f) : 0.f;
        pv[l] = l < H ? __fmaf_rn(b, b, 0.f) : 0.f;
    }
    const float vk = __fmul_rn(fold(pk), inv), vv = __fmul_rn(fold(pv), inv);
    return fuse_score(mode, sk, vk, sv, vv, eps);
}

constexpr int kFuseLanes = 8;   // the lane count score_fuse_kernel uses for up to 8 KV heads

template <int KPT>
__global__ void __launch_bounds__(kCsThreads, 1) select_cluster_kernel(const ClusterSelectParams p) {
    __shared__ int hist[2][256];
    __shared__ int s_warp[kCsWarps];
    __shared__ int s_pub[4];                  // read by the other CTAs of the cluster: [0] equal keys, [1] retained, [2] lowest pruned score
    __shared__ unsigned int s_prefix;
    __shared__ int s_rank, s_count, s_total;
    __shared__ int s_tab[KPT * kCsWarps];     // [chunk][warp] ballot counts of the final sweep
    __shared__ unsigned int s_few[32];        // CTA 0's copy: the last few candidates' keys, appended by the whole cluster
    __shared__ int s_few_n;

    grid_launch_dependents();   // few CTAs: the attention grid may take the other SMs and set up meanwhile
    grid_dependency_wait();
    cg::cluster_group cluster = cg::this_cluster();
    const int n_ranks = (int)cluster.num_blocks(), rank = (int)cluster.block_rank();
    const int b = (int)blockIdx.x / n_ranks, tid = threadIdx.x, S = p.S;
    const int lane = tid & 31, wid = tid >> 5;
    const int t_base = rank * (KPT * kCsThreads);
    const uint8_t* el = p.eligible ? p.eligible + (size_t)b * S : nullptr;
    float* sc = p.score + (size_t)b * S;
    if (tid == 0) s_few_n = 0;                // used at most once, after at least one cluster barrier

    // token of slot i: t_base + i*512 + tid (ascending in (i, tid))
    float sreg[KPT];
    if (p.sim_k) {
        // the similarities of up to four tokens per thread are requested together (one round trip to memory, not one
        // per token and pass), then fused from registers
        constexpr int kBatch = KPT < 4 ? KPT : 4;
#pragma unroll
        for (int i0 = 0; i0 < KPT; i0 += kBatch) {
            float xk[kBatch][8], xv[kBatch][8];
#pragma unroll
            for (int u = 0; u < kBatch; ++u) {
                const int t = t_base + (i0 + u) * kCsThreads + tid;
                const size_t row = ((size_t)b * S + (t < S ? t : 0)) * p.H;
                if (p.vec4) {
#pragma unroll
                    for (int h4 = 0; h4 < 2; ++h4) {
                        float4 a = make_float4(0.f, 0.f, 0.f, 0.f), c = a;
                        if (t < S && h4 * 4 < p.H) {
                            a = __ldg(reinterpret_cast<const float4*>(p.sim_k + row) + h4);
                            c = __ldg(reinterpret_cast<const float4*>(p.sim_v + row) + h4);
                        }
                        xk[u][4 * h4] = a.x; xk[u][4 * h4 + 1] = a.y; xk[u][4 * h4 + 2] = a.z; xk[u][4 * h4 + 3] = a.w;
                        xv[u][4 * h4] = c.x; xv[u][4 * h4 + 1] = c.y; xv[u][4 * h4 + 2] = c.z; xv[u][4 * h4 + 3] = c.w;
                    }
                } else {
#pragma unroll
                    for (int h = 0; h < 8; ++h) {
                        xk[u][h] = (t < S && h < p.H) ? __ldg(p.sim_k + row + h) : 0.f;
                        xv[u][h] = (t < S && h < p.H) ? __ldg(p.sim_v + row + h) : 0.f;
                    }
                }
            }
#pragma unroll
            for (int u = 0; u < kBatch; ++u) sreg[i0 + u] = fuse_token8(xk[u], xv[u], p.H, p.fuse_mode, p.eps);
        }
#pragma unroll
        for (int i = 0; i < KPT; ++i) {
            const int t = t_base + i * kCsThreads + tid;
            if (t < S) {
                sc[t] = sreg[i];
                note_nan_score(p.status, sreg[i], (unsigned long long)b * S + t);
            } else {
                sreg[i] = 0.f;
            }
        }
    } else {
#pragma unroll
        for (int i = 0; i < KPT; ++i) {
            const int t = t_base + i * kCsThreads + tid;
            sreg[i] = t < S ? sc[t] : 0.f;
        }
    }
    auto candidate = [&](int t, float s) -> bool {
        return t >= p.warmup && (el == nullptr || el[t] != 0) && s == s;   // NaN never pruned
    };

    unsigned int key_thr = 0;   // ratio mode: key of the P-th candidate
    int take_eq = 0;            // ratio mode: how many tokens with key == key_thr go (highest index first)
    int n_eq = 0;               // ratio mode: how many candidates have key == key_thr
    float tau = 0.f;
    bool nothing = false;       // nothing to prune

    if (p.mode == TF_SELECT_THRESHOLD) {
        tau = p.threshold[b];
    } else if (p.p_target <= 0) {
        nothing = true;
    } else {
        unsigned int prefix = 0, mask = 0;
        int r = 0, pass = 0;
        for (int shift = 24; shift >= 0; shift -= 8, ++pass) {
            int* h = hist[pass & 1];
            // this buffer was last read by the cluster two passes ago; every CTA has passed the barrier since
            if (tid < 256) h[tid] = 0;
            __syncthreads();
#pragma unroll
            for (int i = 0; i < KPT; ++i) {
                const int t = t_base + i * kCsThreads + tid;
                int bin = 256;   // sentinel: this lane adds nothing
                if (t < S && candidate(t, sreg[i])) {
                    const unsigned int k = score_key(sreg[i]);
                    if ((k & mask) == prefix) bin = (int)((k >> shift) & 255u);
                }
                const unsigned int same = __match_any_sync(0xffffffffu, bin);
                if (bin < 256 && lane == __ffs(same) - 1) atomicAdd(&h[bin], __popc(same));
            }
            cluster.sync();      // every CTA's histogram of this pass is complete
            // descending inclusive scan of the cluster's histogram: the bin where the count reaches r
            int hval = 0, incl = 0;
            if (tid < 256) {
                for (int q = 0; q < n_ranks; ++q) hval += cluster.map_shared_rank(h, q)[255 - tid];
                incl = hval;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int n = __shfl_up_sync(0xffffffffu, incl, o);
                    if (lane >= o) incl += n;
                }
                if (lane == 31) s_warp[wid] = incl;
            }
            __syncthreads();
            if (shift == 24) {   // first pass: the number of candidates E caps the number to prune (same in every CTA)
                int E = 0;
#pragma unroll
                for (int w2 = 0; w2 < 8; ++w2) E += s_warp[w2];
                r = (int)(p.p_target < (long long)E ? p.p_target : (long long)E);
                if (r <= 0) { nothing = true; break; }
            }
            if (tid < 256) {
                int off = 0;
                for (int w2 = 0; w2 < wid; ++w2) off += s_warp[w2];
                incl += off;
                const int excl = incl - hval;
                if (excl < r && incl >= r) {
                    s_prefix = prefix | ((unsigned int)(255 - tid) << shift);
                    s_rank = r - excl;
                    s_count = hval;
                }
            }
            __syncthreads();
            prefix = s_prefix;
            r = s_rank;
            n_eq = s_count;
            mask |= 255u << shift;
            __syncthreads();     // s_warp, s_prefix, s_rank and s_count are written again in the next pass
            // Few candidates left under this prefix (typical after two or three passes): they are collected in CTA 0's
            // shared memory and every CTA ranks them there instead of further histogram passes.  Same result: the key of
            // rank r among them, how many candidates carry it, and the rank within those.  (n_eq is the same in every CTA.)
            if (shift > 0 && n_eq <= 32) {
                unsigned int* few0 = cluster.map_shared_rank(s_few, 0);
                int* few_n0 = cluster.map_shared_rank(&s_few_n, 0);
#pragma unroll
                for (int i = 0; i < KPT; ++i) {
                    const int t = t_base + i * kCsThreads + tid;
                    if (t < S && candidate(t, sreg[i])) {
                        const unsigned int k = score_key(sreg[i]);
                        if ((k & mask) == prefix) few0[atomicAdd(few_n0, 1)] = k;     // exactly n_eq appends in all
                    }
                }
                cluster.sync();
                if (tid < 32) {
                    const unsigned int key = tid < n_eq ? few0[tid] : 0u;
                    int greater = 0, equal = 0;
                    for (int o = 0; o < n_eq; ++o) {
                        const unsigned int ko = __shfl_sync(0xffffffffu, key, o);
                        greater += ko > key ? 1 : 0;
                        equal += ko == key ? 1 : 0;
                    }
                    if (tid < n_eq && greater < r && r <= greater + equal) {   // every lane holding that key writes the same
                        s_prefix = key;
                        s_rank = r - greater;
                        s_count = equal;
                    }
                }
                __syncthreads();
                prefix = s_prefix;
                r = s_rank;
                n_eq = s_count;
                break;
            }
        }
        key_thr = prefix;
        take_eq = r;             // 1 <= r <= n_eq
    }

    // ---- sweep in index order: decide, rank the equal keys, compact ---------------------------------------
    const unsigned int lt = (1u << lane) - 1u;
    auto scan_table = [&]() {    // exclusive prefix over s_tab[0 .. KPT*16), in place; s_total = the sum
        __syncthreads();
        if (wid == 0) {
            constexpr int kEnt = KPT * kCsWarps, kPer = (kEnt + 31) / 32;
            int v[kPer], sum = 0;
#pragma unroll
            for (int e = 0; e < kPer; ++e) { v[e] = lane * kPer + e < kEnt ? s_tab[lane * kPer + e] : 0; sum += v[e]; }
            int incl = sum;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int n = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += n;
            }
            int run = incl - sum;
#pragma unroll
            for (int e = 0; e < kPer; ++e) { if (lane * kPer + e < kEnt) s_tab[lane * kPer + e] = run; run += v[e]; }
            if (lane == 31) s_total = incl;
        }
        __syncthreads();
    };
    unsigned int eq_bits = 0, prune_bits = 0;
#pragma unroll
    for (int i = 0; i < KPT; ++i) {
        const int t = t_base + i * kCsThreads + tid;
        const bool cand = t < S && candidate(t, sreg[i]);
        if (p.mode == TF_SELECT_THRESHOLD) {
            if (cand && sreg[i] > tau) prune_bits |= 1u << i;
        } else if (!nothing && cand) {
            const unsigned int k = score_key(sreg[i]);
            if (k > key_thr) prune_bits |= 1u << i;
            if (k == key_thr) eq_bits |= 1u << i;
        }
    }
    if (p.mode != TF_SELECT_THRESHOLD && !nothing) {          // cluster-uniform
        if (take_eq == n_eq) {
            prune_bits |= eq_bits;                            // every token that ties with the P-th key goes
        } else {
#pragma unroll
            for (int i = 0; i < KPT; ++i) {
                const unsigned int bal = __ballot_sync(0xffffffffu, (eq_bits >> i) & 1u);
                if (lane == 0) s_tab[i * kCsWarps + wid] = __popc(bal);
            }
            scan_table();
            if (tid == 0) s_pub[0] = s_total;
            cluster.sync();
            int eq_before = 0;                                // equal keys in the CTAs before this one
            for (int q = 0; q < rank; ++q) eq_before += cluster.map_shared_rank(s_pub, q)[0];
#pragma unroll
            for (int i = 0; i < KPT; ++i) {
                const bool eq = (eq_bits >> i) & 1u;
                const unsigned int bal = __ballot_sync(0xffffffffu, eq);
                const int eq_rank = eq_before + s_tab[i * kCsWarps + wid] + __popc(bal & lt);   // 0-based among equals, index order
                // the take_eq equals with the highest index: ranks n_eq-take_eq .. n_eq-1
                if (eq && eq_rank >= n_eq - take_eq) prune_bits |= 1u << i;
            }
            __syncthreads();                                  // the table is reused below
        }
    }
    float th_min = CUDART_INF_F;
#pragma unroll
    for (int i = 0; i < KPT; ++i) {
        const int t = t_base + i * kCsThreads + tid;
        const bool keep = t < S && !((prune_bits >> i) & 1u);
        const unsigned int bal = __ballot_sync(0xffffffffu, keep);
        if (lane == 0) s_tab[i * kCsWarps + wid] = __popc(bal);
        if ((prune_bits >> i) & 1u) th_min = fminf(th_min, sreg[i]);
    }
    th_min = -warp_max(-th_min);
    __syncthreads();             // s_warp may still be read by the last radix pass (the nothing-to-prune exit)
    if (lane == 0) s_warp[wid] = __float_as_int(th_min);
    scan_table();
    if (tid == 0) {
        float m = CUDART_INF_F;
        for (int w2 = 0; w2 < kCsWarps; ++w2) m = fminf(m, __int_as_float(s_warp[w2]));
        s_pub[1] = s_total;
        s_pub[2] = __float_as_int(m);
    }
    cluster.sync();
    int kept_before = 0, kept_all = 0;
    for (int q = 0; q < n_ranks; ++q) {
        const int n = cluster.map_shared_rank(s_pub, q)[1];
        kept_before += q < rank ? n : 0;
        kept_all += n;
    }
#pragma unroll
    for (int i = 0; i < KPT; ++i) {
        const int t = t_base + i * kCsThreads + tid;
        const bool in = t < S, keep = in && !((prune_bits >> i) & 1u);
        const unsigned int bal = __ballot_sync(0xffffffffu, keep);
        const int pos = kept_before + s_tab[i * kCsWarps + wid] + __popc(bal & lt);
        if (in) {
            p.keep_mask[(size_t)b * S + t] = keep ? 1 : 0;
            if (keep) p.kept_idx[(size_t)b * S + pos] = t;
            if (t >= kept_all) p.kept_idx[(size_t)b * S + t] = -1;   // the list's tail: positions kept_all .. S-1 (pos <= t, so never a slot just filled)
        }
    }
    if (rank == 0 && tid == 0) {
        p.n_kept[b] = kept_all;
        if (p.theta) {
            float m = CUDART_INF_F;
            for (int q = 0; q < n_ranks; ++q) m = fminf(m, __int_as_float(cluster.map_shared_rank(s_pub, q)[2]));
            p.theta[b] = m;
        }
    }
    cluster.sync();              // nobody leaves while its shared memory may still be read
}

template <int KPT>
cudaError_t launch_form(const ClusterSelectParams& cp, int batch, int n_ranks, cudaStream_t st) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(batch * n_ranks));
    cfg.blockDim = dim3(kCsThreads);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = (unsigned)n_ranks;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, select_cluster_kernel<KPT>, cp);
}

}  // namespace

// Sequence lengths the cluster form takes, and is chosen for: more than 1024 tokens (up to there one CTA per sequence
// is as fast: the cluster's barriers and remote reads cost what the shorter passes save) and at most 8 CTAs x 512
// threads x 8 scores per thread.
bool select_cluster_usable(const tf_shape& s) { return s.seq > 1024 && s.seq <= 8 * kCsThreads * 8; }
bool select_cluster_preferred(const tf_shape& s) { return select_cluster_usable(s); }
bool select_cluster_fuses(const tf_shape& s) { return s.n_kv_heads <= kFuseLanes; }

// sim_k == nullptr: selection only, the scores are read from `score`
cudaError_t launch_select_cluster(tf_ctx* ctx, const tf_shape& s, const tf_filter_params& p, const float* sim_k,
                                  const float* sim_v, float* score, uint8_t* keep_mask, int32_t* kept_idx,
                                  int32_t* n_kept, float* theta, cudaStream_t st) {
    if (!select_cluster_usable(s) || (sim_k && !select_cluster_fuses(s))) return cudaErrorNotSupported;
    if (s.batch == 0) return cudaSuccess;
    ClusterSelectParams cp{};
    cp.sim_k = sim_k; cp.sim_v = sim_v; cp.score = score;
    cp.eligible = p.eligible; cp.threshold = p.threshold;
    cp.S = s.seq; cp.H = s.n_kv_heads; cp.warmup = p.warmup_tokens; cp.mode = p.select_mode; cp.fuse_mode = p.fuse_mode;
    cp.eps = p.var_eps > 0.f ? p.var_eps : 1e-8f;
    cp.vec4 = (sim_k && s.n_kv_heads % 4 == 0 && ((reinterpret_cast<uintptr_t>(sim_k) | reinterpret_cast<uintptr_t>(sim_v)) & 15) == 0) ? 1 : 0;
    cp.p_target = (long long)floor(p.prune_ratio * (double)s.seq);
    cp.keep_mask = keep_mask; cp.kept_idx = kept_idx; cp.n_kept = n_kept; cp.theta = theta;
    cp.status = ctx->dev_status;
    const int n_ranks = s.seq > 2048 ? 8 : 4;
    const int per_rank = (s.seq + n_ranks - 1) / n_ranks;
    int kpt = 1;
    while (kpt * kCsThreads < per_rank) kpt *= 2;
    cudaError_t e = kpt == 1 ? launch_form<1>(cp, s.batch, n_ranks, st) : kpt == 2 ? launch_form<2>(cp, s.batch, n_ranks, st)
                  : kpt == 4 ? launch_form<4>(cp, s.batch, n_ranks, st) : launch_form<8>(cp, s.batch, n_ranks, st);
    ctx->launches += 1;
    return e;
}

}  // namespace tf
