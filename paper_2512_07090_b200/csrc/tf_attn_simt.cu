// Step a5 on CUDA cores: causal (optionally windowed) attention for retained tokens, any dtype.
//
// This is the path fp32 tensors take (fp32 accuracy rules out the 16-bit tensor-core path) and
// the A/B reference for the tensor-core kernel.  One warp owns one (retained token, query head):
// 32 keys at a time, each lane scores one key against the query held in shared memory, the
// warp runs the online softmax, and each lane accumulates 4 output dims over those 32 keys.
// The warp also zeroes the output rows of the pruned tokens that lie between its retained token
// and the previous one (Section 3.2: a skipped token's attention output is zero), so the whole
// of O is written with no separate clearing pass.
#include "tf_common.cuh"

namespace tf {

constexpr int kSimtWarps = 4;

struct AttnParams {
    const void* Q; const void* K; const void* V; void* O;
    Strides3 qs, ks, vs, os;
    int S, Hq, Hkv, window;
    float scale_log2;          // softmax scale * log2(e)
    const int32_t* kept_idx;   // [B,S]
    const int32_t* n_kept;     // [B]
    int retained_only;         // 1: a retained query sees retained tokens' keys / values only
};

template <typename T> __device__ __forceinline__ float to_f(T v);
template <> __device__ __forceinline__ float to_f<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// four consecutive elements (16 bytes of fp32, 8 bytes of bf16; the caller's offset is a multiple of four elements)
__device__ __forceinline__ void load4(const float* p, float (&f)[4]) {
    const float4 v = __ldg(reinterpret_cast<const float4*>(p));
    f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w;
}
__device__ __forceinline__ void load4(const __nv_bfloat16* p, float (&f)[4]) {
    const uint2 v = __ldg(reinterpret_cast<const uint2*>(p));
    f[0] = __uint_as_float(v.x << 16); f[1] = __uint_as_float(v.x & 0xffff0000u);
    f[2] = __uint_as_float(v.y << 16); f[3] = __uint_as_float(v.y & 0xffff0000u);
}

template <typename T>
__device__ __forceinline__ void zero_rows(T* Ob, const Strides3& os, int t_lo, int t_hi, int lane) {
    for (int t = t_lo; t < t_hi; ++t) {
        T* row = Ob + (long long)t * os.t;
#pragma unroll
        for (int i = 0; i < 4; ++i) row[lane * 4 + i] = from_f<T>(0.f);
    }
}

template <typename T>
__global__ void __launch_bounds__(kSimtWarps * 32) attention_simt_kernel(const AttnParams p) {
    constexpr int EPV = Elem<T>::kPerVec;          // elements per 16-byte vector
    constexpr int NVEC = kHeadDim / EPV;
    __shared__ __align__(16) float q_s[kSimtWarps][kHeadDim];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int slot = blockIdx.x * kSimtWarps + warp;   // index into the retained list
    const int qh = blockIdx.y, b = blockIdx.z;
    const int nk = p.n_kept[b];
    if (slot >= max(nk, 1)) return;
    const int32_t* kept = p.kept_idx + (size_t)b * p.S;
    T* Ob = reinterpret_cast<T*>(p.O) + (long long)b * p.os.b + (long long)qh * p.os.h;

    // rows of pruned tokens around this slot
    if (nk == 0) { zero_rows(Ob, p.os, 0, p.S, lane); return; }
    const int t = kept[slot];
    zero_rows(Ob, p.os, slot == 0 ? 0 : kept[slot - 1] + 1, t, lane);
    if (slot == nk - 1) zero_rows(Ob, p.os, t + 1, p.S, lane);

    const int kh = qh / (p.Hq / p.Hkv);
    const T* qrow = reinterpret_cast<const T*>(p.Q) + (long long)b * p.qs.b + (long long)t * p.qs.t + (long long)qh * p.qs.h;
    const T* Kb = reinterpret_cast<const T*>(p.K) + (long long)b * p.ks.b + (long long)kh * p.ks.h;
    const T* Vb = reinterpret_cast<const T*>(p.V) + (long long)b * p.vs.b + (long long)kh * p.vs.h;
#pragma unroll
    for (int i = 0; i < 4; ++i) q_s[warp][lane * 4 + i] = to_f<T>(qrow[lane * 4 + i]) * p.scale_log2;
    __syncwarp();

    // keys are visited by index: token positions, or positions in the retained list (retained_only),
    // where entry c stands for token kept[c] and the query itself is entry `slot`
    const int t_min = (p.window > 0) ? max(0, t - p.window + 1) : 0;
    const int j_hi = p.retained_only ? slot : t;
    const int j_lo = p.retained_only ? first_kept_at_or_after(kept, slot + 1, t_min) : t_min;
    float m = -1e30f, lsum = 0.f, acc[4] = {0.f, 0.f, 0.f, 0.f};
    for (int j0 = j_lo; j0 <= j_hi; j0 += 32) {
        const int j = j0 + lane;
        float s = -1e30f;
        const int tok = (j <= j_hi) ? (p.retained_only ? kept[j] : j) : 0;
        if (j <= j_hi) {
            const T* krow = Kb + (long long)tok * p.ks.t;
            float d0 = 0.f, d1 = 0.f;
#pragma unroll 8
            for (int v = 0; v < NVEC; ++v) {   // eight 16-byte loads in flight per lane: the warp is alone on its row, so
                                               // memory-level parallelism has to come from inside it
                float f[EPV];
                Elem<T>::unpack(ldg16(krow + v * EPV), f);
                const float* qq = &q_s[warp][v * EPV];
#pragma unroll
                for (int e = 0; e < EPV; e += 2) { d0 = fmaf(f[e], qq[e], d0); d1 = fmaf(f[e + 1], qq[e + 1], d1); }
            }
            s = d0 + d1;
        }
        const float m_new = fmaxf(m, warp_max(s));
        const float corr = exp2f(m - m_new);
        const float pj = (j <= j_hi) ? exp2f(s - m_new) : 0.f;
        lsum = lsum * corr + warp_sum(pj);
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[i] *= corr;
        const int n_here = min(32, j_hi - j0 + 1);
        // same order of additions as a plain loop over the block's keys; the value rows of eight keys are requested
        // together (loads first, products after), not one round trip to memory per key
        for (int jj0 = 0; jj0 < n_here; jj0 += 8) {
            float vv[8][4];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int vt = __shfl_sync(0xffffffffu, tok, jj0 + u);
                if (jj0 + u < n_here) load4(Vb + (long long)vt * p.vs.t + lane * 4, vv[u]);
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const float pw = __shfl_sync(0xffffffffu, pj, jj0 + u);
                if (jj0 + u < n_here) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) acc[i] = fmaf(pw, vv[u][i], acc[i]);
                }
            }
        }
        m = m_new;
    }
    const float inv = 1.f / lsum;
    T* orow = Ob + (long long)t * p.os.t;
#pragma unroll
    for (int i = 0; i < 4; ++i) orow[lane * 4 + i] = from_f<T>(acc[i] * inv);
}

cudaError_t launch_attention_simt(tf_ctx* ctx, const tf_shape& s, const tf_filter_params& p,
                                  const void* Q, const void* K, const void* V,
                                  const int32_t* kept_idx, const int32_t* n_kept, void* O,
                                  cudaStream_t st) {
    if (s.batch == 0 || s.seq == 0) return cudaSuccess;
    AttnParams ap{};
    ap.retained_only = (p.kv_visibility == TF_KV_RETAINED);
    ap.Q = Q; ap.K = K; ap.V = V; ap.O = O;
    ap.qs = {s.q_stride[0], s.q_stride[1], s.q_stride[2]};
    ap.ks = {s.k_stride[0], s.k_stride[1], s.k_stride[2]};
    ap.vs = {s.v_stride[0], s.v_stride[1], s.v_stride[2]};
    ap.os = {s.o_stride[0], s.o_stride[1], s.o_stride[2]};
    ap.S = s.seq; ap.Hq = s.n_q_heads; ap.Hkv = s.n_kv_heads; ap.window = s.window;
    const float scale = s.softmax_scale != 0.f ? s.softmax_scale : 1.f / sqrtf((float)s.head_dim);
    ap.scale_log2 = scale * 1.4426950408889634f;
    ap.kept_idx = kept_idx; ap.n_kept = n_kept;
    const dim3 grid((unsigned)((s.seq + kSimtWarps - 1) / kSimtWarps), (unsigned)s.n_q_heads, (unsigned)s.batch);
    if (s.dtype == TF_BF16) attention_simt_kernel<__nv_bfloat16><<<grid, kSimtWarps * 32, 0, st>>>(ap);
    else                    attention_simt_kernel<float><<<grid, kSimtWarps * 32, 0, st>>>(ap);
    ctx->launches += 1;
    ctx->last_attention_kernel = TF_KERNEL_ATTN_SIMT;
    return cudaGetLastError();
}

}  // namespace tf
