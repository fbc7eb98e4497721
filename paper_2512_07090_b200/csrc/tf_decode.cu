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
    float gamma, var_eps, eta;
    double target;                      // the target skip ratio, as the caller gave it
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
    grid_dependency_wait();                 // launched early; the step before this one on the stream must be complete
    const int b = blockIdx.x, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int t = p.pos[b];
    const long long n0 = p.count[b];
    const bool ema = p.anchor_mode == TF_ANCHOR_EMA, incl = p.anchor_mode == TF_ANCHOR_INCL_MEAN;
    const float a = ema ? p.gamma : 1.f, w = ema ? 1.f - p.gamma : 1.f;
    const long long n_cmp = n0 + (incl ? 1 : 0);            // tokens the anchor covers when it is compared
    // the controller's state is read now, under the row loads below, not after the block barrier
    long long steps = 0, skips = 0;
    float tau_old = 0.f;
    if (threadIdx.x == 0) { steps = p.steps[b]; skips = p.skips[b]; tau_old = p.tau[b]; }

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
            // ratio and step in double, the threshold itself is an fp32 state word
            const double rho = steps > 0 ? (double)skips / (double)steps : 0.0;
            const double delta = (double)p.eta * (p.alg1_sign ? (p.target - rho) : (rho - p.target));
            const float tau = tau_old + (float)delta;
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
// serves all G <= 8 query heads of the group, so K and V rows are read once per group.  The two small
// products run on warp-level tensor-core instructions (m16n8k16, bf16 in, fp32 out): the path is
// bandwidth-bound, and the CUDA-core dot products (8 FMAs and 4 shuffles per (head, key)) were what kept
// it from the bandwidth, so the point is the instruction count, not the flops.  Per warp and block of
// 16 keys:
//   S^T[16 keys x 8 heads] = K_blk Q^T     8 products over the 128 dims.  A dot product does not care in
//                                           which order the dims are visited, so lane (g, t) loads 16-byte
//                                           pieces t, t+4, t+8, t+12 of its two key rows (g, g+8) and of
//                                           query head g, and both operands use the same dim order: no
//                                           shared memory, no shuffles, every load a full 16 bytes;
//   online softmax on the accumulator layout (lane holds keys g, g+8 for heads 2t, 2t+1: the maximum
//   over keys is three shuffles); P^T goes back through two 8x8 register transposes (movmatrix);
//   O^T[128 dims x 8 heads] += V_blk^T P^T  8 products.  Lane (g, t) loads dims 16g..16g+15 of its four
//                                           key rows (2t, 2t+1, 2t+8, 2t+9); the pairs "same dim, two
//                                           consecutive keys" the A operand wants are byte permutes.
// The 8 warps take key blocks 8 apart, each with its own online softmax; they are merged through shared
// memory.  With more than one split the CTA leaves (max, sum, unnormalised output) per head in scratch
// and decode_combine_kernel merges the splits.
// ---------------------------------------------------------------------------------------------------
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

__device__ __forceinline__ void mma_bf16_16816(float* d, uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t transpose8x8_b16(uint32_t a) {
    uint32_t d;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
    return d;
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    return (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(lo)) | ((uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(hi)) << 16);
}
__device__ __forceinline__ uint32_t word_of(const uint4& r, int w) { return w == 0 ? r.x : w == 1 ? r.y : w == 2 ? r.z : r.w; }

template <int G>
__global__ void __launch_bounds__(256, 2) decode_attention_gqa_kernel(const DecGqaParams p) {
    __shared__ float part_s[8][G][kPartialFloats];
    grid_dependency_wait();
    const int split = blockIdx.x, kh = blockIdx.y, b = blockIdx.z;
    if (p.skip[b]) {
        if (split == 0 && p.n_splits == 1)
            for (int i = threadIdx.x; i < G * kHeadDim; i += 256)
                p.O[(long long)b * p.o_b + (long long)(kh * G + i / kHeadDim) * p.o_h + (i % kHeadDim)] = __float2bfloat16_rn(0.f);
        return;
    }
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
    const int t_pos = p.pos[b];
    const int j_lo = (p.window > 0) ? max(0, t_pos - p.window + 1) : 0;
    const int n_vis = t_pos - j_lo + 1;
    const int per = ((n_vis + p.n_splits - 1) / p.n_splits + 15) / 16 * 16;     // keys per split, a multiple of 16
    const int k_lo = j_lo + split * per, k_hi = min(t_pos + 1, k_lo + per);       // [k_lo, k_hi)
    const uint4 zero4 = make_uint4(0, 0, 0, 0);

    // Q^T as the B operand of the 8 score products: head g, pieces t + 4i; product 2i + u takes words 2u, 2u + 1
    uint32_t qb[8][2];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const uint4 r = (g < G) ? ldg16(p.Q + (long long)b * p.q_b + (long long)(kh * G + g) * p.q_h + 8 * (t + 4 * i)) : zero4;
        qb[2 * i][0] = r.x; qb[2 * i][1] = r.y; qb[2 * i + 1][0] = r.z; qb[2 * i + 1][1] = r.w;
    }
    const __nv_bfloat16* Kb = p.K + (long long)b * p.ks.b + (long long)kh * p.ks.h;
    const __nv_bfloat16* Vb = p.V + (long long)b * p.vs.b + (long long)kh * p.vs.h + 16 * g;

    // this lane's part of the state: heads 2t and 2t + 1 (m is the same in all lanes of equal t; l is the lane's share)
    float m[2] = {-1e30f, -1e30f}, l[2] = {0.f, 0.f};
    float o[8][4];                                   // O^T: product mt, rows (dims) 16g + mt and 16g + 8 + mt, columns (heads) 2t, 2t + 1
#pragma unroll
    for (int mt = 0; mt < 8; ++mt) { o[mt][0] = o[mt][1] = o[mt][2] = o[mt][3] = 0.f; }

    for (int kb = k_lo + 16 * warp; kb < k_hi; kb += 16 * 8) {       // warp-uniform bounds: the shuffles below name all lanes
        uint4 kr[2][4], vr[4][2];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int j = kb + g + 8 * h;
#pragma unroll
            for (int i = 0; i < 4; ++i) kr[h][i] = (j < k_hi) ? ldg16(Kb + (long long)j * p.ks.t + 8 * (t + 4 * i)) : zero4;
        }
#pragma unroll
        for (int q4 = 0; q4 < 4; ++q4) {
            const int j = kb + 2 * t + (q4 & 1) + 8 * (q4 >> 1);
#pragma unroll
            for (int i = 0; i < 2; ++i) vr[q4][i] = (j < k_hi) ? ldg16(Vb + (long long)j * p.vs.t + 8 * i) : zero4;
        }
        // ---- scores: rows = keys g, g + 8; columns = heads 2t, 2t + 1 -----------------------------------------
        float s[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            mma_bf16_16816(s, kr[0][i].x, kr[1][i].x, kr[0][i].y, kr[1][i].y, qb[2 * i][0], qb[2 * i][1]);
            mma_bf16_16816(s, kr[0][i].z, kr[1][i].z, kr[0][i].w, kr[1][i].w, qb[2 * i + 1][0], qb[2 * i + 1][1]);
        }
        const bool v0 = kb + g < k_hi, v1 = kb + g + 8 < k_hi;
        s[0] = v0 ? s[0] * p.scale_log2 : -1e30f; s[1] = v0 ? s[1] * p.scale_log2 : -1e30f;
        s[2] = v1 ? s[2] * p.scale_log2 : -1e30f; s[3] = v1 ? s[3] * p.scale_log2 : -1e30f;
        float corr[2], pr[4];
#pragma unroll
        for (int c = 0; c < 2; ++c) {
            float mx = fmaxf(s[c], s[c + 2]);
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 4));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 8));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 16));
            const float mn = fmaxf(m[c], mx);
            corr[c] = exp2f(m[c] - mn);
            m[c] = mn;
            pr[c] = v0 ? exp2f(s[c] - mn) : 0.f;
            pr[c + 2] = v1 ? exp2f(s[c + 2] - mn) : 0.f;
            l[c] = fmaf(l[c], corr[c], pr[c] + pr[c + 2]);
        }
        // P^T (keys x heads) -> the B operand wants head g with keys 2t, 2t+1 / 2t+8, 2t+9: two 8x8 transposes
        const uint32_t pb0 = transpose8x8_b16(pack_bf16x2(pr[0], pr[1]));
        const uint32_t pb1 = transpose8x8_b16(pack_bf16x2(pr[2], pr[3]));
#pragma unroll
        for (int mt = 0; mt < 8; ++mt) {
            o[mt][0] *= corr[0]; o[mt][1] *= corr[1]; o[mt][2] *= corr[0]; o[mt][3] *= corr[1];
            const int w = mt >> 1;
            const uint32_t sel = (mt & 1) ? 0x7632u : 0x5410u;     // the high / low halves of two rows' words
            const uint32_t a0 = __byte_perm(word_of(vr[0][0], w), word_of(vr[1][0], w), sel);   // dim 16g + mt,     keys 2t, 2t+1
            const uint32_t a1 = __byte_perm(word_of(vr[0][1], w), word_of(vr[1][1], w), sel);   // dim 16g + 8 + mt, keys 2t, 2t+1
            const uint32_t a2 = __byte_perm(word_of(vr[2][0], w), word_of(vr[3][0], w), sel);   // dim 16g + mt,     keys 2t+8, 2t+9
            const uint32_t a3 = __byte_perm(word_of(vr[2][1], w), word_of(vr[3][1], w), sel);
            mma_bf16_16816(o[mt], a0, a1, a2, a3, pb0, pb1);
        }
    }
    // ---- the lane's share of l -> the sum over the 8 lanes of equal t; then everything into shared memory ---------
#pragma unroll
    for (int c = 0; c < 2; ++c) {
        l[c] += __shfl_xor_sync(0xffffffffu, l[c], 4);
        l[c] += __shfl_xor_sync(0xffffffffu, l[c], 8);
        l[c] += __shfl_xor_sync(0xffffffffu, l[c], 16);
    }
#pragma unroll
    for (int c = 0; c < 2; ++c) {
        const int h = 2 * t + c;
        if (h < G) {
#pragma unroll
            for (int mt = 0; mt < 8; ++mt) {
                part_s[warp][h][16 * g + mt] = o[mt][c];
                part_s[warp][h][16 * g + 8 + mt] = o[mt][c + 2];
            }
            if (g == 0) { part_s[warp][h][kHeadDim] = m[c]; part_s[warp][h][kHeadDim + 1] = l[c]; }
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < G * kHeadDim; i += 256) {
        const int h = i / kHeadDim, d = i % kHeadDim;
        float M = -1e30f;
#pragma unroll
        for (int w2 = 0; w2 < 8; ++w2) M = fmaxf(M, part_s[w2][h][kHeadDim]);
        float L = 0.f, acc = 0.f;
#pragma unroll
        for (int w2 = 0; w2 < 8; ++w2) {
            const float c = exp2f(part_s[w2][h][kHeadDim] - M);
            L = fmaf(part_s[w2][h][kHeadDim + 1], c, L);
            acc = fmaf(part_s[w2][h][d], c, acc);
        }
        const int qh = kh * G + h;
        if (p.n_splits == 1) {
            p.O[(long long)b * p.o_b + (long long)qh * p.o_h + d] = __float2bfloat16_rn(acc / L);
        } else {
            float* dst = p.partial + (((size_t)b * p.Hq + qh) * p.n_splits + split) * kPartialFloats;
            dst[d] = acc;
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
    dp.eta = a.eta; dp.target = p.prune_ratio; dp.alg1_sign = a.alg1_sign;
    dp.sum_k = a.state->sum_k; dp.sum_v = a.state->sum_v; dp.count = reinterpret_cast<long long*>(a.state->count);
    dp.tau = a.state->tau; dp.steps = reinterpret_cast<long long*>(a.state->steps);
    dp.skips = reinterpret_cast<long long*>(a.state->skips);
    dp.score_out = a.score_out; dp.skip_out = a.skip_out; dp.status = ctx->dev_status;
    const size_t smem = 2 * (size_t)s.n_kv_heads * sizeof(float);
    cudaError_t e;
    if (s.dtype == TF_BF16) e = launch_dependent(decode_decide_kernel<__nv_bfloat16>, dim3((unsigned)s.batch), dim3(kDecWarps * 32), smem, st, dp);
    else                    e = launch_dependent(decode_decide_kernel<float>, dim3((unsigned)s.batch), dim3(kDecWarps * 32), smem, st, dp);
    ctx->launches += 1;
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
        // Number of key splits: two CTAs fit an SM, a wave of CTAs costs (a fixed part worth ~192 keys + its keys), and a
        // partly filled wave costs as much as a full one; take the split count with the cheapest estimate, at least
        // 256 keys per split.
        int n_splits = 1;
        {
            const long long groups = (long long)s.batch * s.n_kv_heads, slots = 2ll * sms;
            long long best = -1;
            for (int n = 1; n <= std::max(1, max_keys / 256); ++n) {
                const long long waves = (groups * n + slots - 1) / slots;
                const long long cost = waves * (192 + (max_keys + n - 1) / n);
                if (best < 0 || cost < best) { best = cost; n_splits = n; }
            }
        }
        const size_t need = (size_t)s.batch * s.n_q_heads * n_splits * kPartialFloats * sizeof(float);
        if (n_splits > 1 && (!ctx->workspace || ctx->workspace_bytes < need)) n_splits = 1;
        gp.n_splits = n_splits;
        gp.partial = n_splits > 1 ? static_cast<float*>(ctx->workspace) : nullptr;
        // the partial results overwrite the start of the workspace, where tf_kv_stats keeps its tagged records: the
        // next scan on this workspace clears its region first instead of trusting what it finds there
        if (n_splits > 1) { ctx->scan_user.needs_clear = true; ctx->scan_owned.needs_clear = true; }
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
