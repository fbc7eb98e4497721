// Online decode step: Algorithm 1 for ONE new token per sequence, with the threshold feedback of
// Section 3.3 (T_l <- T_l + eta (P_current - P_tail)) and the attention it gates.
//
// decode_decide_kernel (one CTA per sequence, one warp per KV head at a time):
//   per head: cosine of the current token's key / value to the anchor carried in the state (sum of
//   past tokens, or the EMA of Eq. 1); then one warp: mean / variance over heads, weight alpha
//   (Eq. 2), score s_KV (Eq. 3), threshold adaptation, skip decision; then the anchor takes the
//   token in and the counters advance.  Order as in Algorithm 1: compare first, update after
//   (the inclusive reading updates first).
// decode_attention_kernel (one CTA per (query head, sequence)): standard single-query attention
//   over cache positions <= pos (optionally windowed) unless the token is skipped, in which case
//   its output row is zero (Section 3.2).  The 8 warps take interleaved blocks of 32 keys, each
//   with its own online softmax; the partial results are merged through shared memory.
#include <algorithm>

#include "tf_common.cuh"

namespace tf {

constexpr int kDecWarps = 8;

struct DecideParams {
    const void* K; const void* V;       // cache [B,S,Hkv,128]
    Strides3 ks, vs;
    const int32_t* pos;                 // [B] position of the current token
    int Hkv, anchor_mode, fuse_mode, warmup;
    float gamma, var_eps, eta, target;
    int alg1_sign;
    float* sum_k; float* sum_v; long long* count;      // state
    float* tau; long long* steps; long long* skips;
    float* score_out; uint8_t* skip_out;
    DevStatus* status;
};

template <typename T> __device__ __forceinline__ float dec_to_f(T v);
template <> __device__ __forceinline__ float dec_to_f<float>(float v) { return v; }
template <> __device__ __forceinline__ float dec_to_f<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T dec_from_f(float v);
template <> __device__ __forceinline__ float dec_from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 dec_from_f<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

template <typename T>
__global__ void __launch_bounds__(kDecWarps * 32) decode_decide_kernel(const DecideParams p) {
    extern __shared__ float cos_s[];        // [2][Hkv]
    const int b = blockIdx.x, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int t = p.pos[b];
    const long long n0 = p.count[b];
    const bool ema = p.anchor_mode == TF_ANCHOR_EMA, incl = p.anchor_mode == TF_ANCHOR_INCL_MEAN;
    const float a = ema ? p.gamma : 1.f, w = ema ? 1.f - p.gamma : 1.f;
    const long long n_cmp = n0 + (incl ? 1 : 0);            // tokens the anchor covers when it is compared

    for (int h = warp; h < p.Hkv; h += kDecWarps) {
        const T* kp = reinterpret_cast<const T*>(p.K) + (long long)b * p.ks.b + (long long)t * p.ks.t + (long long)h * p.ks.h + lane * 4;
        const T* vp = reinterpret_cast<const T*>(p.V) + (long long)b * p.vs.b + (long long)t * p.vs.t + (long long)h * p.vs.h + lane * 4;
        float* sk = p.sum_k + ((size_t)b * p.Hkv + h) * kHeadDim + lane * 4;
        float* sv = p.sum_v + ((size_t)b * p.Hkv + h) * kHeadDim + lane * 4;
        float dk = 0.f, kk = 0.f, pk = 0.f, dv = 0.f, vv = 0.f, pv = 0.f;
        float nk4[4], nv4[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float xk = dec_to_f<T>(kp[i]), xv = dec_to_f<T>(vp[i]);
            float ak = sk[i], av = sv[i];
            const float uk = fmaf(a, ak, w * xk), uv = fmaf(a, av, w * xv);    // anchor after the token is taken in
            if (incl) { ak = uk; av = uv; }
            dk = fmaf(xk, ak, dk); kk = fmaf(xk, xk, kk); pk = fmaf(ak, ak, pk);
            dv = fmaf(xv, av, dv); vv = fmaf(xv, xv, vv); pv = fmaf(av, av, pv);
            nk4[i] = uk; nv4[i] = uv;
        }
        dk = warp_sum(dk); kk = warp_sum(kk); pk = warp_sum(pk);
        dv = warp_sum(dv); vv = warp_sum(vv); pv = warp_sum(pv);
        if (lane == 0) {
            float ck = 0.f, cv = 0.f;
            if (n_cmp > 0) {
                const float s = ema ? 1.f : 1.f / (float)n_cmp;     // anchor = sum * s
                ck = (dk * s) / (fmaxf(sqrtf(kk), kNormEps) * fmaxf(sqrtf(pk) * s, kNormEps));
                cv = (dv * s) / (fmaxf(sqrtf(vv), kNormEps) * fmaxf(sqrtf(pv) * s, kNormEps));
            }
            cos_s[h] = ck; cos_s[p.Hkv + h] = cv;
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) { sk[i] = nk4[i]; sv[i] = nv4[i]; }
    }
    __syncthreads();
    if (warp == 0) {
        const int H = p.Hkv;
        float mk = 0.f, mv = 0.f;
        for (int h = lane; h < H; h += 32) { mk += cos_s[h]; mv += cos_s[H + h]; }
        const float inv = 1.f / (float)H;
        mk = warp_sum(mk) * inv; mv = warp_sum(mv) * inv;
        float vk = 0.f, vvv = 0.f;
        for (int h = lane; h < H; h += 32) {
            const float x = cos_s[h] - mk, y = cos_s[H + h] - mv;
            vk = fmaf(x, x, vk); vvv = fmaf(y, y, vvv);
        }
        vk = warp_sum(vk) * inv; vvv = warp_sum(vvv) * inv;
        if (lane == 0) {
            const float eps = p.var_eps;
            float alpha;
            switch (p.fuse_mode) {
                case TF_FUSE_EQ2_LITERAL: alpha = (vk + eps) / (vk + vvv + 2.f * eps); break;
                case TF_FUSE_KEY_ONLY: alpha = 1.f; break;
                case TF_FUSE_VALUE_ONLY: alpha = 0.f; break;
                case TF_FUSE_MEAN: alpha = 0.5f; break;
                default: alpha = (vvv + eps) / (vk + vvv + 2.f * eps); break;
            }
            float s = alpha * mk + (1.f - alpha) * mv;
            s += 0.f;
            const long long steps = p.steps[b], skips = p.skips[b];
            // ratio and step in double, the threshold itself is an fp32 state word
            const double rho = steps > 0 ? (double)skips / (double)steps : 0.0;
            const double delta = (double)p.eta * (p.alg1_sign ? ((double)p.target - rho) : (rho - (double)p.target));
            const float tau = p.tau[b] + (float)delta;
            const bool decide = s > tau;              // false for NaN
            const bool skip = decide && t >= p.warmup;
            p.tau[b] = tau;
            p.steps[b] = steps + 1;
            p.skips[b] = skips + (decide ? 1 : 0);
            p.count[b] = n0 + 1;
            if (p.score_out) p.score_out[b] = s;
            p.skip_out[b] = skip ? 1 : 0;
            if (s != s && p.status) {
                atomicAdd(&p.status->nan_count, 1ull);
                report_error(p.status, TF_ERR_NAN_SCORE, (unsigned long long)b);
            }
        }
    }
}

struct DecAttnParams {
    const void* Q; const void* K; const void* V; void* O;
    long long q_b, q_h, o_b, o_h;       // element strides of the [B,Hq,128] query / output
    Strides3 ks, vs;
    const int32_t* pos; const uint8_t* skip;
    int Hq, Hkv, window;
    float scale_log2;
};

template <typename T>
__global__ void __launch_bounds__(kDecWarps * 32) decode_attention_kernel(const DecAttnParams p) {
    constexpr int EPV = Elem<T>::kPerVec, NVEC = kHeadDim / EPV;
    __shared__ __align__(16) float q_s[kHeadDim];
    __shared__ float m_s[kDecWarps], l_s[kDecWarps];
    __shared__ float acc_s[kDecWarps][kHeadDim];

    grid_dependency_wait();
    const int qh = blockIdx.x, b = blockIdx.y, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    T* orow = reinterpret_cast<T*>(p.O) + (long long)b * p.o_b + (long long)qh * p.o_h;
    if (p.skip[b]) {
        if (threadIdx.x < kHeadDim) orow[threadIdx.x] = dec_from_f<T>(0.f);
        return;
    }
    const int t = p.pos[b];
    const int kh = qh / (p.Hq / p.Hkv);
    const T* qrow = reinterpret_cast<const T*>(p.Q) + (long long)b * p.q_b + (long long)qh * p.q_h;
    if (threadIdx.x < kHeadDim) q_s[threadIdx.x] = dec_to_f<T>(qrow[threadIdx.x]) * p.scale_log2;
    __syncthreads();
    const T* Kb = reinterpret_cast<const T*>(p.K) + (long long)b * p.ks.b + (long long)kh * p.ks.h;
    const T* Vb = reinterpret_cast<const T*>(p.V) + (long long)b * p.vs.b + (long long)kh * p.vs.h;
    const int j_lo = (p.window > 0) ? max(0, t - p.window + 1) : 0;

    float m = -1e30f, lsum = 0.f, acc[4] = {0.f, 0.f, 0.f, 0.f};
    for (int j0 = j_lo + warp * 32; j0 <= t; j0 += kDecWarps * 32) {
        const int j = j0 + lane;
        float s = -1e30f;
        if (j <= t) {
            const T* krow = Kb + (long long)j * p.ks.t;
            float d0 = 0.f, d1 = 0.f;
#pragma unroll 4
            for (int v = 0; v < NVEC; ++v) {
                float f[EPV];
                Elem<T>::unpack(ldg16(krow + v * EPV), f);
                const float* qq = &q_s[v * EPV];
#pragma unroll
                for (int e = 0; e < EPV; e += 2) { d0 = fmaf(f[e], qq[e], d0); d1 = fmaf(f[e + 1], qq[e + 1], d1); }
            }
            s = d0 + d1;
        }
        const float m_new = fmaxf(m, warp_max(s));
        const float corr = exp2f(m - m_new);
        const float pj = (j <= t) ? exp2f(s - m_new) : 0.f;
        lsum = lsum * corr + warp_sum(pj);
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[i] *= corr;
        const int n_here = min(32, t - j0 + 1);
        for (int jj = 0; jj < n_here; ++jj) {
            const float pw = __shfl_sync(0xffffffffu, pj, jj);
            const T* vrow = Vb + (long long)(j0 + jj) * p.vs.t + lane * 4;
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[i] = fmaf(pw, dec_to_f<T>(vrow[i]), acc[i]);
        }
        m = m_new;
    }
    if (lane == 0) { m_s[warp] = m; l_s[warp] = lsum; }
#pragma unroll
    for (int i = 0; i < 4; ++i) acc_s[warp][lane * 4 + i] = acc[i];
    __syncthreads();
    if (threadIdx.x < kHeadDim) {
        float mm = -1e30f;
#pragma unroll
        for (int w2 = 0; w2 < kDecWarps; ++w2) mm = fmaxf(mm, m_s[w2]);
        float l = 0.f, o = 0.f;
#pragma unroll
        for (int w2 = 0; w2 < kDecWarps; ++w2) {
            const float c = exp2f(m_s[w2] - mm);       // a warp that saw no key has l = 0 and acc = 0
            l = fmaf(l_s[w2], c, l);
            o = fmaf(acc_s[w2][threadIdx.x], c, o);
        }
        orow[threadIdx.x] = dec_from_f<T>(o / l);
    }
}

// ---------------------------------------------------------------------------------------------------
// bf16 decode attention for grouped heads: one CTA per (split of the visible keys, KV head, sequence)
// serves all G query heads of the group, so K and V rows are read once per group.  16 lanes share a
// key row (16-byte loads, two adjacent rows per warp instruction); the 16 half-warps of the CTA take
// keys 16 apart, four at a time, each with its own online softmax; half-warps are merged through
// shuffles and shared memory.  With more than one split the CTA leaves (max, sum, unnormalised
// output) per head in scratch and decode_combine_kernel merges the splits.
// ---------------------------------------------------------------------------------------------------
constexpr int kDecBatch = 4;          // keys a half-warp scores before it updates its running maximum
constexpr int kPartialFloats = kHeadDim + 2;

struct DecGqaParams {
    const __nv_bfloat16* Q; const __nv_bfloat16* K; const __nv_bfloat16* V; __nv_bfloat16* O;
    long long q_b, q_h, o_b, o_h;
    Strides3 ks, vs;
    const int32_t* pos; const uint8_t* skip;
    int Hq, Hkv, window, n_splits;
    float scale_log2;
    float* partial;                   // [B][Hq][n_splits][130] when n_splits > 1
};

__device__ __forceinline__ void unpack8(const uint4& r, float* f) {
    f[0] = __uint_as_float(r.x << 16); f[1] = __uint_as_float(r.x & 0xffff0000u);
    f[2] = __uint_as_float(r.y << 16); f[3] = __uint_as_float(r.y & 0xffff0000u);
    f[4] = __uint_as_float(r.z << 16); f[5] = __uint_as_float(r.z & 0xffff0000u);
    f[6] = __uint_as_float(r.w << 16); f[7] = __uint_as_float(r.w & 0xffff0000u);
}

template <int G>
__global__ void __launch_bounds__(256) decode_attention_gqa_kernel(const DecGqaParams p) {
    __shared__ float part_s[8][G][kPartialFloats];
    grid_dependency_wait();
    const int split = blockIdx.x, kh = blockIdx.y, b = blockIdx.z;
    if (p.skip[b]) {
        if (split == 0 && p.n_splits == 1)
            for (int i = threadIdx.x; i < G * kHeadDim; i += 256)
                p.O[(long long)b * p.o_b + (long long)(kh * G + i / kHeadDim) * p.o_h + (i % kHeadDim)] = __float2bfloat16_rn(0.f);
        return;
    }
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, half = lane >> 4, l16 = lane & 15;
    const int t = p.pos[b];
    const int j_lo = (p.window > 0) ? max(0, t - p.window + 1) : 0;
    const int n_vis = t - j_lo + 1;
    const int per = ((n_vis + p.n_splits - 1) / p.n_splits + 15) / 16 * 16;     // keys per split, a multiple of 16
    const int k_lo = j_lo + split * per, k_hi = min(t + 1, k_lo + per);           // [k_lo, k_hi)

    float q[G][8];
#pragma unroll
    for (int h = 0; h < G; ++h) {
        float f[8];
        unpack8(ldg16(p.Q + (long long)b * p.q_b + (long long)(kh * G + h) * p.q_h + l16 * 8), f);
#pragma unroll
        for (int e = 0; e < 8; ++e) q[h][e] = f[e] * p.scale_log2;
    }
    const __nv_bfloat16* Kb = p.K + (long long)b * p.ks.b + (long long)kh * p.ks.h + l16 * 8;
    const __nv_bfloat16* Vb = p.V + (long long)b * p.vs.b + (long long)kh * p.vs.h + l16 * 8;

    float m[G], l[G], acc[G][8];
#pragma unroll
    for (int h = 0; h < G; ++h) {
        m[h] = -1e30f; l[h] = 0.f;
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[h][e] = 0.f;
    }
    // half-warp hw = 2 warp + half takes keys k_lo + hw + 16 i.  The loop bound is the warp's (its lower half-warp's):
    // both halves must make the same number of trips because the shuffles below name all 32 lanes; a key index
    // past the end is handled by the (j < k_hi) predicates.
    for (int kb = k_lo + warp * 2; kb < k_hi; kb += 16 * kDecBatch) {
        const int k0 = kb + half;
        uint4 kr[kDecBatch], vr[kDecBatch];
#pragma unroll
        for (int u = 0; u < kDecBatch; ++u) {
            const int j = k0 + 16 * u;
            kr[u] = (j < k_hi) ? ldg16(Kb + (long long)j * p.ks.t) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int u = 0; u < kDecBatch; ++u) {
            const int j = k0 + 16 * u;
            vr[u] = (j < k_hi) ? ldg16(Vb + (long long)j * p.vs.t) : make_uint4(0, 0, 0, 0);
        }
        float s[G][kDecBatch];
#pragma unroll
        for (int u = 0; u < kDecBatch; ++u) {
            float kf[8];
            unpack8(kr[u], kf);
#pragma unroll
            for (int h = 0; h < G; ++h) {
                float d0 = 0.f, d1 = 0.f;
#pragma unroll
                for (int e = 0; e < 8; e += 2) { d0 = fmaf(q[h][e], kf[e], d0); d1 = fmaf(q[h][e + 1], kf[e + 1], d1); }
                float d = d0 + d1;
#pragma unroll
                for (int o = 8; o > 0; o >>= 1) d += __shfl_xor_sync(0xffffffffu, d, o);   // stays inside the half-warp
                s[h][u] = (k0 + 16 * u < k_hi) ? d : -1e30f;
            }
        }
        float corr[G], pw[G][kDecBatch];
#pragma unroll
        for (int h = 0; h < G; ++h) {
            float mx = m[h];
#pragma unroll
            for (int u = 0; u < kDecBatch; ++u) mx = fmaxf(mx, s[h][u]);
            corr[h] = exp2f(m[h] - mx);
            float ps = 0.f;
#pragma unroll
            for (int u = 0; u < kDecBatch; ++u) {
                pw[h][u] = (k0 + 16 * u < k_hi) ? exp2f(s[h][u] - mx) : 0.f;
                ps += pw[h][u];
            }
            l[h] = fmaf(l[h], corr[h], ps);
            m[h] = mx;
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[h][e] *= corr[h];
        }
#pragma unroll
        for (int u = 0; u < kDecBatch; ++u) {
            float vf[8];
            unpack8(vr[u], vf);
#pragma unroll
            for (int h = 0; h < G; ++h)
#pragma unroll
                for (int e = 0; e < 8; ++e) acc[h][e] = fmaf(pw[h][u], vf[e], acc[h][e]);
        }
    }
    // ---- merge: the two half-warps of a warp by shuffle, the 8 warps through shared memory ---------------
#pragma unroll
    for (int h = 0; h < G; ++h) {
        const float mo = __shfl_xor_sync(0xffffffffu, m[h], 16), lo = __shfl_xor_sync(0xffffffffu, l[h], 16);
        const float mm = fmaxf(m[h], mo);
        const float c_me = exp2f(m[h] - mm), c_ot = exp2f(mo - mm);
        l[h] = l[h] * c_me + lo * c_ot;
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const float ao = __shfl_xor_sync(0xffffffffu, acc[h][e], 16);
            acc[h][e] = acc[h][e] * c_me + ao * c_ot;
        }
        m[h] = mm;
        if (half == 0) {
#pragma unroll
            for (int e = 0; e < 8; ++e) part_s[warp][h][l16 * 8 + e] = acc[h][e];
            if (l16 == 0) { part_s[warp][h][kHeadDim] = m[h]; part_s[warp][h][kHeadDim + 1] = l[h]; }
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < G * kHeadDim; i += 256) {
        const int h = i / kHeadDim, d = i % kHeadDim;
        float M = -1e30f;
#pragma unroll
        for (int w2 = 0; w2 < 8; ++w2) M = fmaxf(M, part_s[w2][h][kHeadDim]);
        float L = 0.f, o = 0.f;
#pragma unroll
        for (int w2 = 0; w2 < 8; ++w2) {
            const float c = exp2f(part_s[w2][h][kHeadDim] - M);
            L = fmaf(part_s[w2][h][kHeadDim + 1], c, L);
            o = fmaf(part_s[w2][h][d], c, o);
        }
        const int qh = kh * G + h;
        if (p.n_splits == 1) {
            p.O[(long long)b * p.o_b + (long long)qh * p.o_h + d] = __float2bfloat16_rn(o / L);
        } else {
            float* dst = p.partial + (((size_t)b * p.Hq + qh) * p.n_splits + split) * kPartialFloats;
            dst[d] = o;
            if (d == 0) { dst[kHeadDim] = M; dst[kHeadDim + 1] = L; }
        }
    }
}

// merges the splits of one (query head, sequence); a skipped token gets its zero row here
__global__ void __launch_bounds__(kHeadDim) decode_combine_kernel(const DecGqaParams p) {
    grid_dependency_wait();
    const int qh = blockIdx.x, b = blockIdx.y, d = threadIdx.x;
    __nv_bfloat16* out = p.O + (long long)b * p.o_b + (long long)qh * p.o_h + d;
    if (p.skip[b]) { *out = __float2bfloat16_rn(0.f); return; }
    const float* src = p.partial + ((size_t)b * p.Hq + qh) * p.n_splits * kPartialFloats;
    float M = -1e30f;
    for (int s2 = 0; s2 < p.n_splits; ++s2) M = fmaxf(M, src[s2 * kPartialFloats + kHeadDim]);
    float L = 0.f, o = 0.f;
    for (int s2 = 0; s2 < p.n_splits; ++s2) {
        const float c = exp2f(src[s2 * kPartialFloats + kHeadDim] - M);
        L = fmaf(src[s2 * kPartialFloats + kHeadDim + 1], c, L);
        o = fmaf(src[s2 * kPartialFloats + d], c, o);
    }
    *out = __float2bfloat16_rn(o / L);
}

cudaError_t launch_decode_step(tf_ctx* ctx, const tf_shape& s, const tf_filter_params& p, const tf_decode_args& a,
                               cudaStream_t st) {
    if (s.batch == 0) return cudaSuccess;
    DecideParams dp{};
    dp.K = a.K_cache; dp.V = a.V_cache;
    dp.ks = {s.k_stride[0], s.k_stride[1], s.k_stride[2]};
    dp.vs = {s.v_stride[0], s.v_stride[1], s.v_stride[2]};
    dp.pos = a.pos; dp.Hkv = s.n_kv_heads; dp.anchor_mode = p.anchor_mode; dp.fuse_mode = p.fuse_mode;
    dp.warmup = p.warmup_tokens; dp.gamma = p.gamma; dp.var_eps = p.var_eps > 0.f ? p.var_eps : 1e-8f;
    dp.eta = a.eta; dp.target = (float)p.prune_ratio; dp.alg1_sign = a.alg1_sign;
    dp.sum_k = a.state->sum_k; dp.sum_v = a.state->sum_v; dp.count = reinterpret_cast<long long*>(a.state->count);
    dp.tau = a.state->tau; dp.steps = reinterpret_cast<long long*>(a.state->steps);
    dp.skips = reinterpret_cast<long long*>(a.state->skips);
    dp.score_out = a.score_out; dp.skip_out = a.skip_out; dp.status = ctx->dev_status;
    const size_t smem = 2 * (size_t)s.n_kv_heads * sizeof(float);
    if (s.dtype == TF_BF16) decode_decide_kernel<__nv_bfloat16><<<s.batch, kDecWarps * 32, smem, st>>>(dp);
    else                    decode_decide_kernel<float><<<s.batch, kDecWarps * 32, smem, st>>>(dp);
    ctx->launches += 1;
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;

    DecAttnParams ap{};
    ap.Q = a.q_new; ap.K = a.K_cache; ap.V = a.V_cache; ap.O = a.O_new;
    ap.q_b = s.q_stride[0]; ap.q_h = s.q_stride[2]; ap.o_b = s.o_stride[0]; ap.o_h = s.o_stride[2];
    ap.ks = dp.ks; ap.vs = dp.vs; ap.pos = a.pos; ap.skip = a.skip_out;
    ap.Hq = s.n_q_heads; ap.Hkv = s.n_kv_heads; ap.window = s.window;
    const float scale = s.softmax_scale != 0.f ? s.softmax_scale : 1.f / sqrtf((float)s.head_dim);
    ap.scale_log2 = scale * 1.4426950408889634f;
    // bf16 with 1, 2, 4 or 8 query heads per KV head: the grouped kernel (K / V read once per group), split
    // over the visible keys when that is needed to fill the GPU and the bound workspace can hold the partials
    const int G = s.n_q_heads / s.n_kv_heads;
    if (s.dtype == TF_BF16 && (G == 1 || G == 2 || G == 4 || G == 8) && (s.q_stride[2] % 8 == 0) && (s.q_stride[0] % 8 == 0) &&
        (reinterpret_cast<uintptr_t>(a.q_new) & 15u) == 0) {
        DecGqaParams gp{};
        gp.Q = static_cast<const __nv_bfloat16*>(a.q_new); gp.K = static_cast<const __nv_bfloat16*>(a.K_cache);
        gp.V = static_cast<const __nv_bfloat16*>(a.V_cache); gp.O = static_cast<__nv_bfloat16*>(a.O_new);
        gp.q_b = ap.q_b; gp.q_h = ap.q_h; gp.o_b = ap.o_b; gp.o_h = ap.o_h;
        gp.ks = ap.ks; gp.vs = ap.vs; gp.pos = a.pos; gp.skip = a.skip_out;
        gp.Hq = s.n_q_heads; gp.Hkv = s.n_kv_heads; gp.window = s.window; gp.scale_log2 = ap.scale_log2;
        int sms = 148;
        { int dev = 0; if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev); }
        const int max_keys = s.window > 0 ? (s.window < s.seq ? s.window : s.seq) : s.seq;   // pos is device data: size for the worst case
        int n_splits = (2 * sms + s.batch * s.n_kv_heads - 1) / (s.batch * s.n_kv_heads);
        n_splits = std::max(1, std::min(n_splits, max_keys / 512));                             // at least 512 keys per split
        const size_t need = (size_t)s.batch * s.n_q_heads * n_splits * kPartialFloats * sizeof(float);
        if (n_splits > 1 && (!ctx->workspace || ctx->workspace_bytes < need)) n_splits = 1;
        gp.n_splits = n_splits;
        gp.partial = n_splits > 1 ? static_cast<float*>(ctx->workspace) : nullptr;
        const dim3 grid((unsigned)n_splits, (unsigned)s.n_kv_heads, (unsigned)s.batch);
        switch (G) {
            case 1: e = launch_dependent(decode_attention_gqa_kernel<1>, grid, dim3(256), 0, st, gp); break;
            case 2: e = launch_dependent(decode_attention_gqa_kernel<2>, grid, dim3(256), 0, st, gp); break;
            case 4: e = launch_dependent(decode_attention_gqa_kernel<4>, grid, dim3(256), 0, st, gp); break;
            default: e = launch_dependent(decode_attention_gqa_kernel<8>, grid, dim3(256), 0, st, gp); break;
        }
        ctx->launches += 1;
        if (e == cudaSuccess && n_splits > 1) {
            e = launch_dependent(decode_combine_kernel, dim3((unsigned)s.n_q_heads, (unsigned)s.batch), dim3(kHeadDim), 0, st, gp);
            ctx->launches += 1;
        }
        return e;
    }
    const dim3 grid((unsigned)s.n_q_heads, (unsigned)s.batch);
    if (s.dtype == TF_BF16) e = launch_dependent(decode_attention_kernel<__nv_bfloat16>, grid, dim3(kDecWarps * 32), 0, st, ap);
    else                    e = launch_dependent(decode_attention_kernel<float>, grid, dim3(kDecWarps * 32), 0, st, ap);
    ctx->launches += 1;
    return e;
}

}  // namespace tf
