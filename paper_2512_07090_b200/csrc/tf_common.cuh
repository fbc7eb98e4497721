// Shared device/host helpers of the Token Filtering CUDA library (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/tf.h"

namespace tf {

constexpr int kHeadDim = 128;
constexpr int kDeviceFlagSlots = 64;       // per-device one-time set-up flags
constexpr float kNormEps = 1e-8f;   // lower clamp of each norm in the cosine

// Device status record: four 64-bit words {code, where, nan_count, reserved}.
struct DevStatus {
    unsigned long long code;
    unsigned long long where;
    unsigned long long nan_count;
    unsigned long long reserved;
};

__device__ __forceinline__ void report_error(DevStatus* st, int code, unsigned long long where) {
    if (st == nullptr) return;
    if (atomicCAS(&st->code, 0ull, (unsigned long long)code) == 0ull) st->where = where;
}

// ---- element access -------------------------------------------------------------------------
// Vec16<T>: one 16-byte global load and its expansion to floats (8 bf16 or 4 fp32).
template <typename T> struct Elem;
template <> struct Elem<float> {
    static constexpr int kPerVec = 4;   // elements per 16-byte vector
    static constexpr int kVecPerLane = 4;  // 16 dims per lane
    __device__ static __forceinline__ void unpack(const uint4& r, float* f) {
        f[0] = __uint_as_float(r.x); f[1] = __uint_as_float(r.y);
        f[2] = __uint_as_float(r.z); f[3] = __uint_as_float(r.w);
    }
};
template <> struct Elem<__nv_bfloat16> {
    static constexpr int kPerVec = 8;
    static constexpr int kVecPerLane = 2;
    // a bf16 is the upper half of the fp32 with the same value
    __device__ static __forceinline__ void unpack(const uint4& r, float* f) {
        f[0] = __uint_as_float(r.x << 16); f[1] = __uint_as_float(r.x & 0xffff0000u);
        f[2] = __uint_as_float(r.y << 16); f[3] = __uint_as_float(r.y & 0xffff0000u);
        f[4] = __uint_as_float(r.z << 16); f[5] = __uint_as_float(r.z & 0xffff0000u);
        f[6] = __uint_as_float(r.w << 16); f[7] = __uint_as_float(r.w & 0xffff0000u);
    }
};

__device__ __forceinline__ uint4 ldg16(const void* p) {
    return __ldg(reinterpret_cast<const uint4*>(p));
}
// streaming 16-byte load: data that is read exactly once should not displace L1 lines
__device__ __forceinline__ uint4 ldg16_stream(const void* p) {
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
    return r;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// first index c in the ascending list kept[0..n) with kept[c] >= target (n if none)
__device__ __forceinline__ int first_kept_at_or_after(const int32_t* kept, int n, int target) {
    int lo = 0, hi = n;
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (kept[mid] < target) lo = mid + 1; else hi = mid;
    }
    return lo;
}

// ---- step a3: mean / population variance over heads, weight alpha (Eq. 2, either reading), fused score (Eq. 3) ----
__device__ __forceinline__ float fuse_alpha(int mode, float var_k, float var_v, float eps) {
    switch (mode) {
        case TF_FUSE_EQ2_LITERAL: return __fdiv_rn(__fadd_rn(var_k, eps), __fmaf_rn(2.f, eps, __fadd_rn(var_k, var_v)));
        case TF_FUSE_KEY_ONLY: return 1.f;
        case TF_FUSE_VALUE_ONLY: return 0.f;
        case TF_FUSE_MEAN: return 0.5f;
        default: return __fdiv_rn(__fadd_rn(var_v, eps), __fmaf_rn(2.f, eps, __fadd_rn(var_k, var_v)));
    }
}
__device__ __forceinline__ float fuse_score(int mode, float mean_k, float var_k, float mean_v, float var_v, float eps) {
    // every rounding is spelled out: the kernels that evaluate this (one launch for step a3 alone, one for a3 + a4)
    // must give the same bits whatever the compiler would contract
    const float alpha = fuse_alpha(mode, var_k, var_v, eps);
    return __fadd_rn(__fmaf_rn(alpha, mean_k, __fmul_rn(__fsub_rn(1.f, alpha), mean_v)), 0.f);   // -0 -> +0
}
__device__ __forceinline__ void note_nan_score(DevStatus* st, float s, unsigned long long token) {
    if (s != s && st) {
        atomicAdd(&st->nan_count, 1ull);
        report_error(st, TF_ERR_NAN_SCORE, token);
    }
}

// ---- step a4: monotone map float -> uint32 (larger score <=> larger key); -0 and +0 share a key ----
__device__ __forceinline__ unsigned int score_key(float s) {
    if (s == 0.f) s = 0.f;
    const unsigned int u = __float_as_uint(s);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float key_score(unsigned int k) {
    const unsigned int u = (k & 0x80000000u) ? (k & 0x7fffffffu) : ~k;
    return __uint_as_float(u);
}

// ---- host-side launch bookkeeping --------------------------------------------------------------
struct Strides3 { long long b, t, h; };

// Launch a kernel that may start while the kernel before it on the stream drains (programmatic
// dependent launch).  Such a kernel executes grid_dependency_wait() before it touches global memory;
// until then only its launch and set-up overlap with its predecessor.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                    Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// Lets the next kernel on the stream (if launched with launch_dependent) become resident now instead of when this
// grid has exited; its grid_dependency_wait() still waits for this grid to complete.  For small grids only: the
// waiting CTAs of the next kernel occupy SM resources.
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

}  // namespace tf

namespace tf {
// Host-side bookkeeping of one scan scratch region (the first section of a workspace).
// The region starts with three counter words {ticket, finished, launches}: every CTA (or worker) of a scan launch
// draws its work from `ticket`; the last CTA to leave the kernel sets ticket and finished back to zero, so a launch
// always starts counting at zero whatever happened to the launch before it (a wait that gave up, workers that stopped
// drawing), and advances `launches`, from which the next launch derives the tag that marks its records as its own.
// Nothing about a launch lives on the host, so a captured launch can be replayed (CUDA graphs) with fresh tags.
struct ScanScratch {
    void* ptr = nullptr;
    size_t capacity = 0;            // bytes the owner of the region provides
    size_t bytes = 0;               // layout key of the records cleared last (0: never cleared)
    bool needs_clear = true;
};
constexpr size_t kScanCounterBytes = 256;   // {ticket, finished} + padding in front of the records

// The tag of this launch's records (never 0, the tag of cleared memory).  Read by every thread that needs it after
// grid_dependency_wait() and BEFORE its CTA calls scan_leave (the last CTA to leave advances the word).
__device__ __forceinline__ unsigned int scan_launch_tag(const unsigned int* counters) {
    const unsigned int n = *reinterpret_cast<const volatile unsigned int*>(counters + 2);
    return n == 0xffffffffu ? 1u : n + 1u;
}
// Drawn by one thread per CTA / worker after grid_dependency_wait().
__device__ __forceinline__ unsigned int scan_draw_ticket(unsigned int* counters) { return atomicAdd(counters, 1u); }
// Called by one thread per CTA when the CTA will draw no more tickets (and its threads have read the launch tag);
// n_ctas = gridDim.x.
__device__ __forceinline__ void scan_leave(unsigned int* counters, unsigned int n_ctas) {
    __threadfence();
    if (atomicAdd(counters + 1, 1u) == n_ctas - 1u) {
        atomicExch(counters, 0u);
        atomicExch(counters + 1, 0u);
        const unsigned int n = *reinterpret_cast<volatile unsigned int*>(counters + 2);
        atomicExch(counters + 2, n == 0xffffffffu ? 1u : n + 1u);
    }
}
}  // namespace tf

// The opaque context of include/tf.h.
struct tf_ctx {
    int device;
    tf::DevStatus* dev_status;     // device memory, 4 words
    void* workspace;               // caller-owned
    size_t workspace_bytes;
    tf::ScanScratch scan_user;     // scan bookkeeping of the caller's workspace
    tf::ScanScratch scan_owned;    // ... and of owned_ws
    int use_tensor_cores;          // bf16 attention path
    int scan_path;                 // tf_kv_stats: 0 = choose, 1 = plain CUDA-core kernel, 2 / 3 = Gram-matrix kernel, one tile per CTA / persistent
    int select_form;               // selection: 0 = choose by sequence length, 1 = one CTA per sequence, 2 = a cluster per sequence
    int attention_form;            // tensor-core kernel: 0 = choose by shape and grid size, 1 = shared K/V tiles (two row tiles), 2 = split K/V tiles, 3 = single, 4 / 5 = shared K/V tiles (two / four query heads of a KV group)
    long long launches;            // kernels launched through this context
    int last_scan_kernel;          // TF_KERNEL_* of the latest similarity scan / attention launched through this context
    int last_attention_kernel;
    long long max_polls;           // bounded waits (tf_set_wait_limits): polls of a look-back record, < 0 = default
    long long wait_cycles;         // ... and clock cycles of an mbarrier wait, < 0 = default
    // tf_layer_filter_host staging (owned, grown on demand)
    void* stage;
    size_t stage_bytes;
    void* owned_ws;
    size_t owned_ws_bytes;
    // ... its copy-in and copy-out streams and the events that chain them with the caller's stream
    static constexpr int kHostEvents = 3 + 2 * 8;
    bool host_streams_ready;
    cudaStream_t s_in, s_out;
    cudaEvent_t ev[kHostEvents];
};

namespace tf {
constexpr int kDefaultMaxPolls = 1 << 20;              // >= 32 ns apart plus an L2 round trip each: of the order of a second
constexpr long long kDefaultWaitCycles = 1000000000ll; // ~0.5 s
inline int ctx_max_polls(const tf_ctx* c) { return c->max_polls >= 0 ? (int)(c->max_polls > 0x7fffffff ? 0x7fffffff : c->max_polls) : kDefaultMaxPolls; }
inline long long ctx_wait_cycles(const tf_ctx* c) { return c->wait_cycles >= 0 ? c->wait_cycles : kDefaultWaitCycles; }
}  // namespace tf

// ---- per-kernel launchers (defined in the .cu files, called by tf_api.cu) ----------------------
namespace tf {

struct ScanPlan {            // how tf_kv_stats tiles a shape
    int chunk_tokens;        // tokens per CTA tile
    int n_chains;            // batch * n_kv_heads
    int n_chunks;            // ceil(seq / chunk_tokens)
    size_t agg_offset, prefix_offset;   // byte offsets of the record arrays in the scratch
    size_t bytes;            // scratch bytes (ticket word + records), 256-aligned
};
ScanPlan scan_plan(const tf_shape& s);
size_t gram_scratch_bytes(const tf_shape& s);   // records of the Gram-matrix kernels (bf16), counters included
// what tf_kv_stats may need for this shape whichever kernel it picks
inline size_t scan_scratch_bytes(const tf_shape& s) {
    const size_t a = scan_plan(s).bytes, b = s.dtype == TF_BF16 ? gram_scratch_bytes(s) : 0;
    return a > b ? a : b;
}

cudaError_t launch_kv_stats(tf_ctx* ctx, const tf_shape& s, const tf_filter_params& p,
                            const void* K, const void* V, float* sim_k, float* sim_v,
                            const tf_carry* carry, ScanScratch* scan_scratch, cudaStream_t st);
// bf16 running-sum anchors through 128-token Gram matrices on the tensor cores (tf_scan_tc.cu)
bool kv_stats_gram_usable(const tf_shape& s, const tf_filter_params& p);
cudaError_t launch_kv_stats_gram(tf_ctx* ctx, const tf_shape& s, const tf_filter_params& p,
                                 const void* K, const void* V, float* sim_k, float* sim_v,
                                 const tf_carry* carry, ScanScratch* scan_scratch, cudaStream_t st);
cudaError_t launch_score_fuse(tf_ctx* ctx, const tf_shape& s, const tf_filter_params& p,
                              const float* sim_k, const float* sim_v, float* score, cudaStream_t st);
cudaError_t launch_select(tf_ctx* ctx, const tf_shape& s, const tf_filter_params& p,
                          const float* score, uint8_t* keep_mask, int32_t* kept_idx,
                          int32_t* n_kept, float* theta, cudaStream_t st);
// steps a3 + a4 by a thread-block cluster per sequence (tf_select_cluster.cu); sim_k == nullptr: a4 alone on `score`
bool select_cluster_usable(const tf_shape& s);      // sequence lengths it can take
bool select_cluster_preferred(const tf_shape& s);   // ... and those it is chosen for
bool select_cluster_fuses(const tf_shape& s);       // step a3 inside the same launch (up to 8 KV heads)
cudaError_t launch_select_cluster(tf_ctx* ctx, const tf_shape& s, const tf_filter_params& p, const float* sim_k,
                                  const float* sim_v, float* score, uint8_t* keep_mask, int32_t* kept_idx,
                                  int32_t* n_kept, float* theta, cudaStream_t st);
// a3 then a4: one launch where the cluster form takes the sequence length, else the two kernels
cudaError_t launch_score_select(tf_ctx* ctx, const tf_shape& s, const tf_filter_params& p, const float* sim_k,
                                const float* sim_v, float* score, uint8_t* keep_mask, int32_t* kept_idx,
                                int32_t* n_kept, float* theta, cudaStream_t st);
cudaError_t launch_attention_simt(tf_ctx* ctx, const tf_shape& s, const tf_filter_params& p,
                                  const void* Q, const void* K, const void* V,
                                  const int32_t* kept_idx, const int32_t* n_kept, void* O,
                                  cudaStream_t st);
struct tf_decode_args {
    const void* q_new; const void* K_cache; const void* V_cache; const int32_t* pos;
    const tf_decode_state* state; void* O_new; float* score_out; uint8_t* skip_out;
    float eta; int alg1_sign;
};
cudaError_t launch_decode_step(tf_ctx* ctx, const tf_shape& s, const tf_filter_params& p, const tf_decode_args& a,
                               cudaStream_t st);
// returns cudaErrorNotSupported when the tensor-core path cannot take this call
// kv_compact: TF_KV_RETAINED only -- device scratch of kv_compact_bytes(s) bytes for the retained
// tokens' keys and values
cudaError_t launch_attention_tc(tf_ctx* ctx, const tf_shape& s, const tf_filter_params& p,
                                const void* Q, const void* K, const void* V,
                                const int32_t* kept_idx, const int32_t* n_kept, void* O,
                                void* kv_compact, cudaStream_t st);
size_t kv_compact_bytes(const tf_shape& s);
// marks the built-in scratch array of tf_kv_stats_static on `device` for clearing before its next use
void static_scratch_invalidate(int device);

}  // namespace tf
