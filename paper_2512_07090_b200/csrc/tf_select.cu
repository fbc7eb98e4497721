// Step a4: keep/prune selection and compaction, one CTA per sequence.
//
// RATIO mode prunes exactly P = min(E, floor(ratio*S)) eligible tokens: those that come first
// when eligible tokens are ordered by (score descending, index descending).  The P-th key is
// found with a 4-pass, 8-bit MSB-first radix select over order-preserving 32-bit keys; tokens
// whose key equals it are then taken from the highest index down.  THRESHOLD mode prunes the
// eligible tokens whose score is strictly above threshold[b] (Alg. 1, "skip if s_KV > tau").
// The retained positions are compacted in ascending order with warp ballots and a block-wide
// prefix sum.  For sequences of up to 16384 tokens every thread keeps its scores in registers
// (token i*1024 + tid in slot i), so the passes run out of registers and shared memory; longer
// sequences stage the scores in shared memory (up to 51200 tokens) or re-read them from global memory
// on each pass.  (Producing the scores inside this
// kernel as well was measured: one CTA per sequence reads the per-head similarities far too slowly.)
#include <math_constants.h>

#include "tf_common.cuh"

namespace tf {

constexpr int kSelThreads = 1024;
constexpr int kSelWarps = kSelThreads / 32;
constexpr int kMaxTableChunks = 64;   // longer sequences (> 65536 tokens) fall back to two block scans per 1024 tokens

struct SelectParams {
    const float* score;        // [B,S]
    const uint8_t* eligible;   // [B,S] or null
    const float* threshold;    // [B] (threshold mode)
    int S, warmup, mode;
    long long p_target;        // floor(ratio*S), computed on the host in double
    int stage;                 // re-reading form only: 1 = the launch has S floats of dynamic shared memory for the scores
    uint8_t* keep_mask; int32_t* kept_idx; int32_t* n_kept; float* theta;
};

// block-wide exclusive prefix over one flag per thread; returns this thread's exclusive rank
// and the block total (s_warp must hold kSelWarps ints; two barriers inside)
__device__ __forceinline__ int block_rank(bool flag, int* s_warp, int& total) {
    const unsigned int bal = __ballot_sync(0xffffffffu, flag);
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    if (lane == 0) s_warp[wid] = __popc(bal);
    __syncthreads();
    int before = 0, tot = 0;
#pragma unroll
    for (int w2 = 0; w2 < kSelWarps; ++w2) {
        const int c = s_warp[w2];
        before += (w2 < wid) ? c : 0;
        tot += c;
    }
    __syncthreads();
    total = tot;
    return before + __popc(bal & ((1u << lane) - 1u));
}

// KPT = scores per thread held in registers (0: read them from global memory each time)
template <int KPT>
__global__ void __launch_bounds__(kSelThreads, 1) select_kernel(const SelectParams p) {
    __shared__ int hist[256];
    __shared__ int s_warp[kSelWarps];
    __shared__ unsigned int s_prefix;
    __shared__ int s_rank, s_count, s_few_eq, s_total;
    __shared__ int s_tab[KPT > 0 ? KPT : kMaxTableChunks][kSelWarps];   // [chunk][warp] ballot counts of the final sweep
    __shared__ unsigned int s_few[32];

    grid_launch_dependents();   // one CTA per sequence: the attention grid may take the other SMs and set up meanwhile
    grid_dependency_wait();
    const int b = blockIdx.x, tid = threadIdx.x, S = p.S;
    const float* sc = p.score + (size_t)b * S;
    if (KPT == 0 && p.stage) {   // too many scores for registers: the passes below read them from shared memory
        extern __shared__ float s_scores[];
        for (int t = tid; t < S; t += kSelThreads) s_scores[t] = sc[t];
        __syncthreads();
        sc = s_scores;
    }
    const uint8_t* el = p.eligible ? p.eligible + (size_t)b * S : nullptr;
    constexpr int NR = KPT > 0 ? KPT : 1;
    float sreg[NR];
    if (KPT > 0) {
#pragma unroll
        for (int i = 0; i < NR; ++i) {
            const int t = i * kSelThreads + tid;
            float s = 0.f;
            if (t < S) {
                s = sc[t];
            }
            sreg[i] = s;
        }
    }
    // score of token t = i*1024 + tid (i is a compile-time index wherever KPT > 0)
    auto score_at = [&](int i, int t) -> float { return KPT > 0 ? sreg[KPT > 0 ? i : 0] : sc[t]; };
    constexpr int kChunks = KPT;   // register form: exactly KPT chunks of 1024 tokens
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
    } else {
        if (p.p_target <= 0) {
            nothing = true;
        } else {
            // radix select: rank r (1-based from the top) among candidates matching the prefix so far.  The number
            // of candidates E, which caps the number to prune (P = min(E, target)), is the total of the first pass's
            // histogram.
            unsigned int prefix = 0, mask = 0;
            int r = 0;
            for (int shift = 24; shift >= 0; shift -= 8) {
                for (int i = tid; i < 256; i += kSelThreads) hist[i] = 0;
                __syncthreads();
#pragma unroll
                for (int i = 0; i < (KPT > 0 ? kChunks : 1 << 30); ++i) {
                    const int t0 = i * kSelThreads;
                    if (KPT == 0 && t0 >= S) break;
                    const int t = t0 + tid;
                    int bin = 256;   // sentinel: this lane adds nothing
                    if (t < S) {
                        const float s = score_at(i, t);
                        if (candidate(t, s)) {
                            const unsigned int k = score_key(s);
                            if ((k & mask) == prefix) bin = (int)((k >> shift) & 255u);
                        }
                    }
                    // scores crowd into a few bins: one shared-memory atomic per distinct bin per warp
                    const unsigned int same = __match_any_sync(0xffffffffu, bin);
                    if (bin < 256 && (tid & 31) == __ffs(same) - 1) atomicAdd(&hist[bin], __popc(same));
                }
                __syncthreads();
                // descending inclusive scan of the histogram: the bin where the count reaches r
                int hval = 0, incl = 0;
                if (tid < 256) {
                    hval = hist[255 - tid];
                    incl = hval;
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const int n = __shfl_up_sync(0xffffffffu, incl, o);
                        if ((tid & 31) >= o) incl += n;
                    }
                    if ((tid & 31) == 31) s_warp[tid >> 5] = incl;
                }
                __syncthreads();
                if (shift == 24) {                       // first pass: E is known now (uniform over the CTA)
                    int E = 0;
#pragma unroll
                    for (int w2 = 0; w2 < 8; ++w2) E += s_warp[w2];
                    r = (int)(p.p_target < (long long)E ? p.p_target : (long long)E);
                    if (r <= 0) { nothing = true; break; }
                }
                if (tid < 256) {
                    int off = 0;
                    for (int w2 = 0; w2 < (tid >> 5); ++w2) off += s_warp[w2];
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
                // (no barrier here: the next pass writes s_prefix, s_rank and s_count only after two more barriers)
                // Few candidates left under this prefix (typical after two passes: scores share their exponent): one
                // warp ranks them directly instead of two more histogram passes.  Same result: the key of rank r among
                // them, how many candidates carry it, and the rank within those.
                if (shift > 0 && n_eq <= 32) {
                    __syncthreads();                          // everybody has read s_count
                    if (tid == 0) s_count = 0;
                    __syncthreads();
#pragma unroll
                    for (int i = 0; i < (KPT > 0 ? kChunks : 1 << 30); ++i) {
                        const int t0 = i * kSelThreads;
                        if (KPT == 0 && t0 >= S) break;
                        const int t = t0 + tid;
                        if (t < S) {
                            const float sv = score_at(i, t);
                            if (candidate(t, sv)) {
                                const unsigned int k = score_key(sv);
                                if ((k & mask) == prefix) s_few[atomicAdd(&s_count, 1)] = k;
                            }
                        }
                    }
                    __syncthreads();
                    if (tid < 32) {
                        const unsigned int key = tid < n_eq ? s_few[tid] : 0u;
                        int greater = 0, equal = 0;
                        for (int o = 0; o < n_eq; ++o) {
                            const unsigned int ko = __shfl_sync(0xffffffffu, key, o);
                            greater += ko > key ? 1 : 0;
                            equal += ko == key ? 1 : 0;
                        }
                        if (tid < n_eq && greater < r && r <= greater + equal) {   // every lane holding that key writes the same
                            s_prefix = key;
                            s_rank = r - greater;
                            s_few_eq = equal;
                        }
                    }
                    __syncthreads();
                    prefix = s_prefix;
                    r = s_rank;
                    n_eq = s_few_eq;
                    break;
                }
            }
            key_thr = prefix;
            take_eq = r;   // 1 <= r <= n_eq
        }
    }

    // ---- sweep in index order: decide, count equals, compact ---------------------------------------
    int kept_base = 0, eq_base = 0;
    float th_min = CUDART_INF_F;
    if constexpr (KPT > 0) {
        // Register form: ranks in index order (token = chunk * 1024 + thread) come from ONE block-wide scan of a
        // [chunk][warp] table of ballot counts per question (rank among the equal keys, position among the kept
        // tokens), instead of two block scans per chunk of 1024 tokens.
        int* tab = &s_tab[0][0];
        const int lane = tid & 31, wid = tid >> 5;
        const unsigned int lt = (1u << lane) - 1u;
        auto scan_table = [&]() {          // exclusive prefix over tab[0 .. KPT*32), in place; s_total = the sum
            __syncthreads();
            if (wid == 0) {
                int v[NR], sum = 0;
#pragma unroll
                for (int e = 0; e < NR; ++e) { v[e] = tab[lane * NR + e]; sum += v[e]; }
                int incl = sum;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int n = __shfl_up_sync(0xffffffffu, incl, o);
                    if (lane >= o) incl += n;
                }
                int run = incl - sum;
#pragma unroll
                for (int e = 0; e < NR; ++e) { tab[lane * NR + e] = run; run += v[e]; }
                if (lane == 31) s_total = incl;
            }
            __syncthreads();
        };
        unsigned int eq_bits = 0, prune_bits = 0;
#pragma unroll
        for (int i = 0; i < NR; ++i) {
            const int t = i * kSelThreads + tid;
            const float sv = sreg[i];
            const bool cand = t < S && candidate(t, sv);
            if (p.mode == TF_SELECT_THRESHOLD) {
                if (cand && sv > tau) prune_bits |= 1u << i;
            } else if (!nothing && cand) {
                const unsigned int k = score_key(sv);
                if (k > key_thr) prune_bits |= 1u << i;
                if (k == key_thr) eq_bits |= 1u << i;
            }
        }
        if (p.mode != TF_SELECT_THRESHOLD && !nothing) {      // CTA-uniform
#pragma unroll
            for (int i = 0; i < NR; ++i) {
                const unsigned int bal = __ballot_sync(0xffffffffu, (eq_bits >> i) & 1u);
                if (lane == 0) tab[i * kSelWarps + wid] = __popc(bal);
            }
            scan_table();
#pragma unroll
            for (int i = 0; i < NR; ++i) {
                const bool eq = (eq_bits >> i) & 1u;
                const unsigned int bal = __ballot_sync(0xffffffffu, eq);
                const int eq_rank = tab[i * kSelWarps + wid] + __popc(bal & lt);     // 0-based among equals, index order
                // the take_eq equals with the highest index: ranks n_eq-take_eq .. n_eq-1
                if (eq && eq_rank >= n_eq - take_eq) prune_bits |= 1u << i;
            }
            __syncthreads();                                   // the table is reused below
        }
#pragma unroll
        for (int i = 0; i < NR; ++i) {
            const int t = i * kSelThreads + tid;
            const bool keep = t < S && !((prune_bits >> i) & 1u);
            const unsigned int bal = __ballot_sync(0xffffffffu, keep);
            if (lane == 0) tab[i * kSelWarps + wid] = __popc(bal);
        }
        scan_table();
#pragma unroll
        for (int i = 0; i < NR; ++i) {
            const int t = i * kSelThreads + tid;
            const bool in = t < S, prune = (prune_bits >> i) & 1u;
            const bool keep = in && !prune;
            const unsigned int bal = __ballot_sync(0xffffffffu, keep);
            const int pos = tab[i * kSelWarps + wid] + __popc(bal & lt);
            if (prune) th_min = fminf(th_min, sreg[i]);
            if (in) {
                p.keep_mask[(size_t)b * S + t] = keep ? 1 : 0;
                if (keep) p.kept_idx[(size_t)b * S + pos] = t;
            }
        }
        kept_base = s_total;
    } else if ((S + kSelThreads - 1) / kSelThreads <= kMaxTableChunks) {
        // The same one-scan-per-question sweep with a run-time number of chunks: the per-chunk decisions are kept as bits
        // of two 64-bit words per thread, the scores are read again (shared or global memory) where they are needed.
        const int n_chunks = (S + kSelThreads - 1) / kSelThreads;
        int* tab = &s_tab[0][0];
        const int lane = tid & 31, wid = tid >> 5;
        const unsigned int lt = (1u << lane) - 1u;
        auto scan_table = [&]() {          // exclusive prefix over tab[0 .. n_chunks*32), in place; s_total = the sum
            __syncthreads();
            if (wid == 0) {
                int sum = 0;
                for (int e = 0; e < n_chunks; ++e) sum += tab[lane * n_chunks + e];
                int incl = sum;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int n = __shfl_up_sync(0xffffffffu, incl, o);
                    if (lane >= o) incl += n;
                }
                int run = incl - sum;
                for (int e = 0; e < n_chunks; ++e) { const int v = tab[lane * n_chunks + e]; tab[lane * n_chunks + e] = run; run += v; }
                if (lane == 31) s_total = incl;
            }
            __syncthreads();
        };
        unsigned long long eq_bits = 0ull, prune_bits = 0ull;
        for (int i = 0; i < n_chunks; ++i) {
            const int t = i * kSelThreads + tid;
            const float sv = t < S ? sc[t] : 0.f;
            const bool cand = t < S && candidate(t, sv);
            if (p.mode == TF_SELECT_THRESHOLD) {
                if (cand && sv > tau) prune_bits |= 1ull << i;
            } else if (!nothing && cand) {
                const unsigned int k = score_key(sv);
                if (k > key_thr) prune_bits |= 1ull << i;
                if (k == key_thr) eq_bits |= 1ull << i;
            }
        }
        if (p.mode != TF_SELECT_THRESHOLD && !nothing) {      // CTA-uniform
            for (int i = 0; i < n_chunks; ++i) {
                const unsigned int bal = __ballot_sync(0xffffffffu, (eq_bits >> i) & 1ull);
                if (lane == 0) tab[i * kSelWarps + wid] = __popc(bal);
            }
            scan_table();
            for (int i = 0; i < n_chunks; ++i) {
                const bool eq = (eq_bits >> i) & 1ull;
                const unsigned int bal = __ballot_sync(0xffffffffu, eq);
                const int eq_rank = tab[i * kSelWarps + wid] + __popc(bal & lt);     // 0-based among equals, index order
                if (eq && eq_rank >= n_eq - take_eq) prune_bits |= 1ull << i;        // the take_eq equals with the highest index
            }
            __syncthreads();                                   // the table is reused below
        }
        for (int i = 0; i < n_chunks; ++i) {
            const int t = i * kSelThreads + tid;
            const bool keep = t < S && !((prune_bits >> i) & 1ull);
            const unsigned int bal = __ballot_sync(0xffffffffu, keep);
            if (lane == 0) tab[i * kSelWarps + wid] = __popc(bal);
        }
        scan_table();
        for (int i = 0; i < n_chunks; ++i) {
            const int t = i * kSelThreads + tid;
            const bool in = t < S, prune = (prune_bits >> i) & 1ull;
            const bool keep = in && !prune;
            const unsigned int bal = __ballot_sync(0xffffffffu, keep);
            const int pos = tab[i * kSelWarps + wid] + __popc(bal & lt);
            if (prune) th_min = fminf(th_min, sc[t]);
            if (in) {
                p.keep_mask[(size_t)b * S + t] = keep ? 1 : 0;
                if (keep) p.kept_idx[(size_t)b * S + pos] = t;
            }
        }
        kept_base = s_total;
    } else {
    #pragma unroll
        for (int i = 0; i < (KPT > 0 ? kChunks : 1 << 30); ++i) {
            const int t0 = i * kSelThreads;
            if (t0 >= S) break;
            const int t = t0 + tid;
            const bool in = t < S;
            const float s = in ? score_at(i, t) : 0.f;
            const bool cand = in && candidate(t, s);
            bool prune = false;
            if (p.mode == TF_SELECT_THRESHOLD) {
                prune = cand && (s > tau);
            } else if (!nothing) {
                const unsigned int k = cand ? score_key(s) : 0u;
                const bool eq = cand && (k == key_thr);
                int eq_tot;
                const int eq_rank = block_rank(eq, s_warp, eq_tot) + eq_base;   // 0-based among equals
                eq_base += eq_tot;
                // the take_eq equals with the highest index: ranks n_eq-take_eq .. n_eq-1
                prune = cand && ((k > key_thr) || (eq && eq_rank >= n_eq - take_eq));
            }
            if (prune) th_min = fminf(th_min, s);
            const bool keep = in && !prune;
            int kept_tot;
            const int pos = block_rank(keep, s_warp, kept_tot) + kept_base;
            kept_base += kept_tot;
            if (in) {
                p.keep_mask[(size_t)b * S + t] = keep ? 1 : 0;
                if (keep) p.kept_idx[(size_t)b * S + pos] = t;
            }
        }
    }
    for (int i = kept_base + tid; i < S; i += kSelThreads) p.kept_idx[(size_t)b * S + i] = -1;
    if (tid == 0) p.n_kept[b] = kept_base;
    if (p.theta) {
        // lowest pruned score
        th_min = -warp_max(-th_min);
        if ((tid & 31) == 0) s_warp[tid >> 5] = __float_as_int(th_min);
        __syncthreads();
        if (tid == 0) {
            float m = CUDART_INF_F;
            for (int w2 = 0; w2 < kSelWarps; ++w2) m = fminf(m, __int_as_float(s_warp[w2]));
            p.theta[b] = m;
        }
    }
}

namespace {
cudaError_t launch_select_form(const SelectParams& sp, int batch, cudaStream_t st) {
    const dim3 grid(batch), block(kSelThreads);
    const int S = sp.S;
    if (S <= 2 * kSelThreads) return launch_dependent(select_kernel<2>, grid, block, 0, st, sp);
    if (S <= 4 * kSelThreads) return launch_dependent(select_kernel<4>, grid, block, 0, st, sp);
    if (S <= 8 * kSelThreads) return launch_dependent(select_kernel<8>, grid, block, 0, st, sp);
    if (S <= 16 * kSelThreads) return launch_dependent(select_kernel<16>, grid, block, 0, st, sp);
    // longer sequences: the scores go to shared memory once (up to 200 KiB = 51200 tokens), else every pass re-reads them
    constexpr size_t kStageMax = 200 << 10;
    SelectParams sp2 = sp;
    const size_t need = (size_t)S * sizeof(float);
    sp2.stage = need <= kStageMax ? 1 : 0;
    if (sp2.stage) {
        static bool attr_set_dev[kDeviceFlagSlots] = {};
        int dev = 0;
        cudaGetDevice(&dev);
        bool& attr_set = attr_set_dev[dev >= 0 && dev < kDeviceFlagSlots ? dev : 0];
        if (!attr_set) {
            cudaError_t e = cudaFuncSetAttribute(select_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kStageMax);
            if (e != cudaSuccess) return e;
            attr_set = true;
        }
    }
    return launch_dependent(select_kernel<0>, grid, block, sp2.stage ? need : 0, st, sp2);
}
}  // namespace

cudaError_t launch_select(tf_ctx* ctx, const tf_shape& s, const tf_filter_params& p,
                          const float* score, uint8_t* keep_mask, int32_t* kept_idx,
                          int32_t* n_kept, float* theta, cudaStream_t st) {
    if (s.batch == 0) return cudaSuccess;
    // sequences of 1025 to 32768 tokens are shared by the CTAs of a cluster
    if (ctx->select_form == 2 || (ctx->select_form == 0 && select_cluster_preferred(s)))
        return launch_select_cluster(ctx, s, p, nullptr, nullptr, const_cast<float*>(score), keep_mask, kept_idx, n_kept, theta, st);
    SelectParams sp{};
    sp.score = score; sp.eligible = p.eligible; sp.threshold = p.threshold;
    sp.S = s.seq; sp.warmup = p.warmup_tokens; sp.mode = p.select_mode;
    sp.p_target = (long long)floor(p.prune_ratio * (double)s.seq);
    sp.keep_mask = keep_mask; sp.kept_idx = kept_idx; sp.n_kept = n_kept; sp.theta = theta;
    cudaError_t e = launch_select_form(sp, s.batch, st);
    ctx->launches += 1;
    return e;
}

cudaError_t launch_score_select(tf_ctx* ctx, const tf_shape& s, const tf_filter_params& p, const float* sim_k,
                                const float* sim_v, float* score, uint8_t* keep_mask, int32_t* kept_idx,
                                int32_t* n_kept, float* theta, cudaStream_t st) {
    if ((ctx->select_form == 2 && select_cluster_usable(s) && select_cluster_fuses(s)) ||
        (ctx->select_form == 0 && select_cluster_preferred(s) && select_cluster_fuses(s)))
        return launch_select_cluster(ctx, s, p, sim_k, sim_v, score, keep_mask, kept_idx, n_kept, theta, st);
    cudaError_t e = launch_score_fuse(ctx, s, p, sim_k, sim_v, score, st);
    if (e == cudaSuccess) e = launch_select(ctx, s, p, score, keep_mask, kept_idx, n_kept, theta, st);
    return e;
}

}  // namespace tf
