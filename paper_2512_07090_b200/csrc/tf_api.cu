// C-ABI entry points of include/tf.h: argument checks, workspace carving, kernel sequencing.
// Every step of the layer runs in the kernels of this library; there is no host fallback.
#include <math.h>
#include <new>
#include <string.h>

#include "tf_common.cuh"

namespace {

using namespace tf;

inline size_t align256(size_t x) { return (x + 255) / 256 * 256; }

// Sections of the caller's workspace.
struct WsLayout {
    size_t scan, sim_k, sim_v, score, keep_mask, kept_idx, n_kept, theta, kv_compact, total;
};

WsLayout ws_layout(const tf_shape& s, const tf_filter_params* p) {
    WsLayout w{};
    const size_t tokens = (size_t)s.batch * (size_t)s.seq;
    size_t off = 0;
    w.scan = off;      off += scan_scratch_bytes(s);   // whichever scan kernel gets picked
    w.sim_k = off;     off += align256(tokens * s.n_kv_heads * sizeof(float));
    w.sim_v = off;     off += align256(tokens * s.n_kv_heads * sizeof(float));
    w.score = off;     off += align256(tokens * sizeof(float));
    w.keep_mask = off; off += align256(tokens);
    w.kept_idx = off;  off += align256(tokens * sizeof(int32_t));
    w.n_kept = off;    off += align256((size_t)s.batch * sizeof(int32_t));
    w.theta = off;     off += align256((size_t)s.batch * sizeof(float));
    w.kv_compact = off;   // retained tokens' K and V (TF_KV_RETAINED on the tensor-core path only)
    if (p && p->kv_visibility == TF_KV_RETAINED && s.dtype == TF_BF16) off += kv_compact_bytes(s);
    w.total = off;
    return w;
}

bool stride_ok(const int64_t st[3], int dtype) {
    const int64_t m = (dtype == TF_BF16) ? 8 : 4;   // 16-byte vectors
    return st[0] % m == 0 && st[1] % m == 0 && st[2] % m == 0 && st[1] > 0 && st[2] > 0 && st[0] >= 0;
}
bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

tf_status check_shape(const tf_shape* s) {
    if (!s) return TF_ERR_INVALID_ARG;
    if (s->batch < 0 || s->seq < 0 || s->n_q_heads <= 0 || s->n_kv_heads <= 0) return TF_ERR_INVALID_ARG;
    if (s->n_q_heads % s->n_kv_heads != 0) return TF_ERR_INVALID_ARG;
    if (s->window < 0 || !(s->softmax_scale >= 0.f)) return TF_ERR_INVALID_ARG;
    if (s->head_dim != kHeadDim) return TF_ERR_UNSUPPORTED;
    if (s->dtype != TF_F32 && s->dtype != TF_BF16) return TF_ERR_UNSUPPORTED;
    if ((long long)s->batch * s->seq > (1ll << 31) - 1) return TF_ERR_UNSUPPORTED;
    if (s->batch > 65535 || s->n_q_heads > 65535) return TF_ERR_UNSUPPORTED;
    return TF_OK;
}

tf_status check_params(const tf_filter_params* p) {
    if (!p) return TF_ERR_INVALID_ARG;
    if (!(p->prune_ratio >= 0.0 && p->prune_ratio < 1.0)) return TF_ERR_INVALID_ARG;
    if (p->warmup_tokens < 0) return TF_ERR_INVALID_ARG;
    if (p->anchor_mode < TF_ANCHOR_PAST_MEAN || p->anchor_mode > TF_ANCHOR_EMA) return TF_ERR_INVALID_ARG;
    if (p->anchor_mode == TF_ANCHOR_EMA && !(p->gamma > 0.f && p->gamma < 1.f)) return TF_ERR_INVALID_ARG;
    if (p->fuse_mode < TF_FUSE_INVVAR || p->fuse_mode > TF_FUSE_MEAN) return TF_ERR_INVALID_ARG;
    if (p->select_mode != TF_SELECT_RATIO && p->select_mode != TF_SELECT_THRESHOLD) return TF_ERR_INVALID_ARG;
    if (p->select_mode == TF_SELECT_THRESHOLD && p->threshold == nullptr) return TF_ERR_INVALID_ARG;
    if (p->kv_visibility != TF_KV_ALL && p->kv_visibility != TF_KV_RETAINED) return TF_ERR_INVALID_ARG;
    if (!(p->var_eps >= 0.f)) return TF_ERR_INVALID_ARG;
    return TF_OK;
}

tf_status check_kv(const tf_shape* s, const void* K, const void* V) {
    if (!K || !V) return TF_ERR_INVALID_ARG;
    if (!aligned16(K) || !aligned16(V)) return TF_ERR_UNSUPPORTED;
    if (!stride_ok(s->k_stride, s->dtype) || !stride_ok(s->v_stride, s->dtype)) return TF_ERR_UNSUPPORTED;
    return TF_OK;
}

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
        target = dev;
    }
    ~DeviceGuard() { if (prev >= 0 && prev != target) cudaSetDevice(prev); }
    int target = -1;
};

// NotSupported is how a launcher says "this call is outside what my kernel takes"
tf_status to_status(cudaError_t e) {
    return e == cudaSuccess ? TF_OK : (e == cudaErrorNotSupported ? TF_ERR_UNSUPPORTED : TF_ERR_CUDA);
}

// after a bounded wait gave up, or a launch failed, the records of every scan scratch this context knows are suspect
void invalidate_scan_scratch(tf_ctx* ctx) {
    ctx->scan_user.needs_clear = true;
    ctx->scan_owned.needs_clear = true;
    tf::static_scratch_invalidate(ctx->device);
}

// kv_compact: TF_KV_RETAINED on the tensor-core path only -- kv_compact_bytes(shape of the WHOLE call) bytes in the
// bound workspace (a call on a group of heads reuses the front of it)
tf_status attention_dispatch(tf_ctx* ctx, const tf_shape& s, const tf_filter_params& p, const void* Q,
                             const void* K, const void* V, const int32_t* kept_idx,
                             const int32_t* n_kept, void* O, void* kv_compact, cudaStream_t st) {
    if (s.dtype == TF_BF16 && ctx->use_tensor_cores) {
        const cudaError_t e = launch_attention_tc(ctx, s, p, Q, K, V, kept_idx, n_kept, O, kv_compact, st);
        // The default path falls back to the CUDA-core kernel only when no tensor map can describe the caller's
        // layout; an explicitly requested form is a requirement, and any other failure is an error.
        if (e != cudaErrorNotSupported || ctx->attention_form != 0) return to_status(e);
    }
    return to_status(launch_attention_simt(ctx, s, p, Q, K, V, kept_idx, n_kept, O, st));
}

// the workspace section for the retained tokens' K / V, or nullptr when this call does not need one
tf_status kv_compact_section(tf_ctx* ctx, const tf_shape& s, const tf_filter_params& p, void** out) {
    *out = nullptr;
    if (p.kv_visibility != TF_KV_RETAINED || s.dtype != TF_BF16 || !ctx->use_tensor_cores) return TF_OK;
    const WsLayout w = ws_layout(s, &p);
    if (!ctx->workspace || ctx->workspace_bytes < w.total) return TF_ERR_WORKSPACE;
    *out = static_cast<char*>(ctx->workspace) + w.kv_compact;
    return TF_OK;
}

}  // namespace

extern "C" {

void tf_default_params(tf_filter_params* p) {
    if (!p) return;
    memset(p, 0, sizeof(*p));
    p->prune_ratio = 0.5;
    p->warmup_tokens = 1;
    p->anchor_mode = TF_ANCHOR_PAST_MEAN;
    p->gamma = 0.9f;
    p->fuse_mode = TF_FUSE_INVVAR;
    p->var_eps = 1e-8f;
    p->select_mode = TF_SELECT_RATIO;
    p->kv_visibility = TF_KV_ALL;
}

tf_status tf_create(tf_ctx** out, int device) {
    if (!out) return TF_ERR_INVALID_ARG;
    *out = nullptr;
    int n = 0;
    if (cudaGetDeviceCount(&n) != cudaSuccess || device < 0 || device >= n) return TF_ERR_CUDA;
    DeviceGuard g(device);
    if (!g.ok) return TF_ERR_CUDA;
    tf_ctx* c = new (std::nothrow) tf_ctx{};
    if (!c) return TF_ERR_CUDA;
    c->device = device;
    c->use_tensor_cores = 1;
    c->max_polls = -1;
    c->wait_cycles = -1;
    if (cudaMalloc(reinterpret_cast<void**>(&c->dev_status), sizeof(DevStatus)) != cudaSuccess ||
        cudaMemset(c->dev_status, 0, sizeof(DevStatus)) != cudaSuccess) {
        delete c;
        return TF_ERR_CUDA;
    }
    *out = c;
    return TF_OK;
}

tf_status tf_destroy(tf_ctx* ctx) {
    if (!ctx) return TF_OK;
    DeviceGuard g(ctx->device);
    if (ctx->dev_status) cudaFree(ctx->dev_status);
    if (ctx->stage) cudaFree(ctx->stage);
    if (ctx->owned_ws) cudaFree(ctx->owned_ws);
    if (ctx->host_streams_ready) {
        cudaStreamDestroy(ctx->s_in);
        cudaStreamDestroy(ctx->s_out);
        for (int i = 0; i < tf_ctx::kHostEvents; ++i) cudaEventDestroy(ctx->ev[i]);
    }
    delete ctx;
    return TF_OK;
}

tf_status tf_workspace_bytes(const tf_shape* shape, const tf_filter_params* params, size_t* bytes) {
    if (!bytes) return TF_ERR_INVALID_ARG;
    tf_status s = check_shape(shape);
    if (s != TF_OK) return s;
    *bytes = ws_layout(*shape, params).total;
    return TF_OK;
}

tf_status tf_set_workspace(tf_ctx* ctx, void* device_ptr, size_t bytes) {
    if (!ctx) return TF_ERR_INVALID_ARG;
    if (device_ptr && (reinterpret_cast<uintptr_t>(device_ptr) & 255u)) return TF_ERR_INVALID_ARG;
    ctx->workspace = device_ptr;
    ctx->workspace_bytes = device_ptr ? bytes : 0;
    ctx->scan_user = tf::ScanScratch();
    ctx->scan_user.ptr = device_ptr;
    ctx->scan_user.capacity = ctx->workspace_bytes;
    return TF_OK;
}

tf_status tf_kv_stats(tf_ctx* ctx, const tf_shape* shape, const tf_filter_params* params,
                      const void* K, const void* V, float* sim_k, float* sim_v,
                      const tf_carry* carry, void* stream) {
    if (!ctx) return TF_ERR_INVALID_ARG;
    tf_status s = check_shape(shape);
    if (s == TF_OK) s = check_params(params);
    if (s == TF_OK) s = check_kv(shape, K, V);
    if (s != TF_OK) return s;
    if (!sim_k || !sim_v) return TF_ERR_INVALID_ARG;
    if (!ctx->workspace || ctx->workspace_bytes < scan_scratch_bytes(*shape)) return TF_ERR_WORKSPACE;
    DeviceGuard g(ctx->device);
    if (!g.ok) return TF_ERR_CUDA;
    return to_status(launch_kv_stats(ctx, *shape, *params, K, V, sim_k, sim_v, carry, &ctx->scan_user,
                                     static_cast<cudaStream_t>(stream)));
}

tf_status tf_score_fuse(tf_ctx* ctx, const tf_shape* shape, const tf_filter_params* params,
                        const float* sim_k, const float* sim_v, float* score, void* stream) {
    if (!ctx) return TF_ERR_INVALID_ARG;
    tf_status s = check_shape(shape);
    if (s == TF_OK) s = check_params(params);
    if (s != TF_OK) return s;
    if (!sim_k || !sim_v || !score) return TF_ERR_INVALID_ARG;
    DeviceGuard g(ctx->device);
    if (!g.ok) return TF_ERR_CUDA;
    cudaError_t e = launch_score_fuse(ctx, *shape, *params, sim_k, sim_v, score, static_cast<cudaStream_t>(stream));
    return to_status(e);
}

tf_status tf_select(tf_ctx* ctx, const tf_shape* shape, const tf_filter_params* params,
                    const float* score, uint8_t* keep_mask, int32_t* kept_idx, int32_t* n_kept,
                    float* theta, void* stream) {
    if (!ctx) return TF_ERR_INVALID_ARG;
    tf_status s = check_shape(shape);
    if (s == TF_OK) s = check_params(params);
    if (s != TF_OK) return s;
    if (!score || !keep_mask || !kept_idx || !n_kept) return TF_ERR_INVALID_ARG;
    DeviceGuard g(ctx->device);
    if (!g.ok) return TF_ERR_CUDA;
    cudaError_t e = launch_select(ctx, *shape, *params, score, keep_mask, kept_idx, n_kept, theta,
                                  static_cast<cudaStream_t>(stream));
    return to_status(e);
}

tf_status tf_score_select(tf_ctx* ctx, const tf_shape* shape, const tf_filter_params* params,
                          const float* sim_k, const float* sim_v, float* score, uint8_t* keep_mask,
                          int32_t* kept_idx, int32_t* n_kept, float* theta, void* stream) {
    if (!ctx) return TF_ERR_INVALID_ARG;
    tf_status s = check_shape(shape);
    if (s == TF_OK) s = check_params(params);
    if (s != TF_OK) return s;
    if (!sim_k || !sim_v || !score || !keep_mask || !kept_idx || !n_kept) return TF_ERR_INVALID_ARG;
    DeviceGuard g(ctx->device);
    if (!g.ok) return TF_ERR_CUDA;
    return to_status(launch_score_select(ctx, *shape, *params, sim_k, sim_v, score, keep_mask, kept_idx, n_kept, theta,
                                         static_cast<cudaStream_t>(stream)));
}

tf_status tf_pruned_attention(tf_ctx* ctx, const tf_shape* shape, const tf_filter_params* params,
                              const void* Q, const void* K, const void* V,
                              const int32_t* kept_idx, const int32_t* n_kept, void* O, void* stream) {
    if (!ctx) return TF_ERR_INVALID_ARG;
    tf_status s = check_shape(shape);
    if (s == TF_OK) s = check_params(params);
    if (s == TF_OK) s = check_kv(shape, K, V);
    if (s != TF_OK) return s;
    if (!Q || !O || !kept_idx || !n_kept) return TF_ERR_INVALID_ARG;
    if (!aligned16(Q) || !aligned16(O)) return TF_ERR_UNSUPPORTED;
    if (!stride_ok(shape->q_stride, shape->dtype) || !stride_ok(shape->o_stride, shape->dtype)) return TF_ERR_UNSUPPORTED;
    DeviceGuard g(ctx->device);
    if (!g.ok) return TF_ERR_CUDA;
    void* kv_compact = nullptr;
    s = kv_compact_section(ctx, *shape, *params, &kv_compact);
    if (s != TF_OK) return s;
    return attention_dispatch(ctx, *shape, *params, Q, K, V, kept_idx, n_kept, O, kv_compact, static_cast<cudaStream_t>(stream));
}

tf_status tf_layer_filter(tf_ctx* ctx, const tf_shape* shape, const tf_filter_params* params,
                          const void* Q, const void* K, const void* V, void* O,
                          float* score, uint8_t* keep_mask, int32_t* kept_idx, int32_t* n_kept,
                          void* stream) {
    if (!ctx) return TF_ERR_INVALID_ARG;
    tf_status s = check_shape(shape);
    if (s == TF_OK) s = check_params(params);
    if (s == TF_OK) s = check_kv(shape, K, V);
    if (s != TF_OK) return s;
    if (!Q || !O) return TF_ERR_INVALID_ARG;
    if (!aligned16(Q) || !aligned16(O)) return TF_ERR_UNSUPPORTED;
    if (!stride_ok(shape->q_stride, shape->dtype) || !stride_ok(shape->o_stride, shape->dtype)) return TF_ERR_UNSUPPORTED;
    const WsLayout w = ws_layout(*shape, params);
    if (!ctx->workspace || ctx->workspace_bytes < w.total) return TF_ERR_WORKSPACE;
    DeviceGuard g(ctx->device);
    if (!g.ok) return TF_ERR_CUDA;
    char* ws = static_cast<char*>(ctx->workspace);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    float* sim_k = reinterpret_cast<float*>(ws + w.sim_k);
    float* sim_v = reinterpret_cast<float*>(ws + w.sim_v);
    if (!score) score = reinterpret_cast<float*>(ws + w.score);
    if (!keep_mask) keep_mask = reinterpret_cast<uint8_t*>(ws + w.keep_mask);
    if (!kept_idx) kept_idx = reinterpret_cast<int32_t*>(ws + w.kept_idx);
    if (!n_kept) n_kept = reinterpret_cast<int32_t*>(ws + w.n_kept);
    float* theta = reinterpret_cast<float*>(ws + w.theta);

    ScanScratch* scan = (ctx->workspace == ctx->owned_ws && ctx->owned_ws) ? &ctx->scan_owned : &ctx->scan_user;
    cudaError_t e = launch_kv_stats(ctx, *shape, *params, K, V, sim_k, sim_v, nullptr, scan, st);
    if (e == cudaSuccess) e = launch_score_select(ctx, *shape, *params, sim_k, sim_v, score, keep_mask, kept_idx, n_kept, theta, st);
    if (e != cudaSuccess) return to_status(e);
    void* kv_compact = nullptr;
    s = kv_compact_section(ctx, *shape, *params, &kv_compact);
    if (s != TF_OK) return s;
    return attention_dispatch(ctx, *shape, *params, Q, K, V, kept_idx, n_kept, O, kv_compact, st);
}

tf_status tf_layer_filter_host(tf_ctx* ctx, const tf_shape* shape, const tf_filter_params* params,
                               const void* Q_host, const void* K_host, const void* V_host,
                               void* O_host, float* score_host, uint8_t* keep_mask_host,
                               int32_t* kept_idx_host, int32_t* n_kept_host, void* stream) {
    if (!ctx) return TF_ERR_INVALID_ARG;
    tf_status s = check_shape(shape);
    if (s == TF_OK) s = check_params(params);
    if (s != TF_OK) return s;
    if (!Q_host || !K_host || !V_host || !O_host) return TF_ERR_INVALID_ARG;
    if (params->eligible || params->threshold) return TF_ERR_UNSUPPORTED;   // those stay device pointers
    const size_t es = shape->dtype == TF_BF16 ? 2 : 4;
    const int64_t d = kHeadDim;
    // dense token-major only
    const int64_t qd[3] = {(int64_t)shape->seq * shape->n_q_heads * d, (int64_t)shape->n_q_heads * d, d};
    const int64_t kd[3] = {(int64_t)shape->seq * shape->n_kv_heads * d, (int64_t)shape->n_kv_heads * d, d};
    for (int i = 0; i < 3; ++i)
        if (shape->q_stride[i] != qd[i] || shape->o_stride[i] != qd[i] || shape->k_stride[i] != kd[i] ||
            shape->v_stride[i] != kd[i])
            return TF_ERR_UNSUPPORTED;
    DeviceGuard g(ctx->device);
    if (!g.ok) return TF_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t tokens = (size_t)shape->batch * shape->seq;
    const size_t qb = align256(tokens * shape->n_q_heads * d * es), kb = align256(tokens * shape->n_kv_heads * d * es);
    const size_t sb = align256(tokens * 4), mb = align256(tokens), ib = align256(tokens * 4), nb = align256((size_t)shape->batch * 4);
    const size_t need = 2 * qb + 2 * kb + sb + mb + ib + nb;
    if (ctx->stage_bytes < need) {
        if (ctx->stage) { cudaStreamSynchronize(st); cudaFree(ctx->stage); ctx->stage = nullptr; ctx->stage_bytes = 0; }
        if (cudaMalloc(&ctx->stage, need) != cudaSuccess) return TF_ERR_CUDA;
        ctx->stage_bytes = need;
    }
    const WsLayout w = ws_layout(*shape, params);
    if (ctx->owned_ws_bytes < w.total) {
        if (ctx->owned_ws) { cudaStreamSynchronize(st); cudaFree(ctx->owned_ws); ctx->owned_ws = nullptr; ctx->owned_ws_bytes = 0; }
        if (cudaMalloc(&ctx->owned_ws, w.total) != cudaSuccess) return TF_ERR_CUDA;
        ctx->owned_ws_bytes = w.total;
        ctx->scan_owned = tf::ScanScratch();
        ctx->scan_owned.ptr = ctx->owned_ws;
        ctx->scan_owned.capacity = ctx->owned_ws_bytes;
    }
    char* base = static_cast<char*>(ctx->stage);
    char* dQ = base; char* dO = base + qb; void* dK = base + 2 * qb; void* dV = base + 2 * qb + kb;
    float* dS = reinterpret_cast<float*>(base + 2 * qb + 2 * kb);
    uint8_t* dM = reinterpret_cast<uint8_t*>(base + 2 * qb + 2 * kb + sb);
    int32_t* dI = reinterpret_cast<int32_t*>(base + 2 * qb + 2 * kb + sb + mb);
    int32_t* dN = reinterpret_cast<int32_t*>(base + 2 * qb + 2 * kb + sb + mb + ib);

    // Pipeline over the two directions of the host link: K and V go first (the filter needs all of them and no
    // Q), then Q arrives in groups of query heads while the attention of the group before runs and its output
    // rows travel back.  Copies in: one internal stream; kernels: the caller's stream; copies out: a second
    // internal stream; events chain them.
    if (!ctx->host_streams_ready) {
        if (cudaStreamCreateWithFlags(&ctx->s_in, cudaStreamNonBlocking) != cudaSuccess ||
            cudaStreamCreateWithFlags(&ctx->s_out, cudaStreamNonBlocking) != cudaSuccess)
            return TF_ERR_CUDA;
        for (int i = 0; i < tf_ctx::kHostEvents; ++i)
            if (cudaEventCreateWithFlags(&ctx->ev[i], cudaEventDisableTiming) != cudaSuccess) return TF_ERR_CUDA;
        ctx->host_streams_ready = true;
    }
    const int gqa = shape->n_q_heads / shape->n_kv_heads;
    int groups = 1;                                           // head groups of whole KV-head groups, >= 2 MB of Q each
    for (int g2 : {8, 4, 2})
        if (groups == 1 && shape->n_q_heads % g2 == 0 && (shape->n_q_heads / g2) % gqa == 0 &&
            tokens * (size_t)(shape->n_q_heads / g2) * d * es >= ((size_t)2 << 20))
            groups = g2;
    const int hq_g = shape->n_q_heads / groups, hkv_g = shape->n_kv_heads / groups;
    cudaEvent_t ev_start = ctx->ev[0], ev_kv = ctx->ev[1], ev_sel = ctx->ev[2];
    cudaError_t e = cudaEventRecord(ev_start, st);             // whatever the caller queued before is done first
    if (e == cudaSuccess) e = cudaStreamWaitEvent(ctx->s_in, ev_start, 0);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(ctx->s_out, ev_start, 0);
    if (e == cudaSuccess) e = cudaMemcpyAsync(dK, K_host, tokens * shape->n_kv_heads * d * es, cudaMemcpyHostToDevice, ctx->s_in);
    if (e == cudaSuccess) e = cudaMemcpyAsync(dV, V_host, tokens * shape->n_kv_heads * d * es, cudaMemcpyHostToDevice, ctx->s_in);
    if (e == cudaSuccess) e = cudaEventRecord(ev_kv, ctx->s_in);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(st, ev_kv, 0);
    if (e != cudaSuccess) return TF_ERR_CUDA;

    void* saved_ws = ctx->workspace; const size_t saved_bytes = ctx->workspace_bytes;
    ctx->workspace = ctx->owned_ws; ctx->workspace_bytes = ctx->owned_ws_bytes;
    {   // steps a1-a4 on the device copies (the same launches tf_layer_filter makes)
        char* ws = static_cast<char*>(ctx->workspace);
        float* sim_k = reinterpret_cast<float*>(ws + w.sim_k);
        float* sim_v = reinterpret_cast<float*>(ws + w.sim_v);
        float* theta = reinterpret_cast<float*>(ws + w.theta);
        tf_shape ds = *shape;                                  // device copies are dense like the host tensors
        e = launch_kv_stats(ctx, ds, *params, dK, dV, sim_k, sim_v, nullptr, &ctx->scan_owned, st);
        if (e == cudaSuccess) e = launch_score_select(ctx, ds, *params, sim_k, sim_v, dS, dM, dI, dN, theta, st);
        if (e == cudaSuccess) e = cudaEventRecord(ev_sel, st);
    }
    s = to_status(e);
    void* kv_compact = nullptr;                                // the whole call's section: every head group reuses its front
    if (s == TF_OK) s = kv_compact_section(ctx, *shape, *params, &kv_compact);
    const size_t row = (size_t)shape->n_q_heads * d * es, row_g = (size_t)hq_g * d * es;   // bytes per token: all heads / one group
    for (int g2 = 0; g2 < groups && s == TF_OK; ++g2) {
        cudaEvent_t ev_q = ctx->ev[3 + 2 * g2], ev_att = ctx->ev[4 + 2 * g2];
        const size_t off = (size_t)g2 * row_g;
        e = cudaMemcpy2DAsync(dQ + off, row, static_cast<const char*>(Q_host) + off, row, row_g, tokens, cudaMemcpyHostToDevice, ctx->s_in);
        if (e == cudaSuccess) e = cudaEventRecord(ev_q, ctx->s_in);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(st, ev_q, 0);
        if (e != cudaSuccess) { s = TF_ERR_CUDA; break; }
        tf_shape gs = *shape;                                  // this group's heads: same strides, fewer heads, shifted bases
        gs.n_q_heads = hq_g; gs.n_kv_heads = hkv_g;
        const size_t kv_off = (size_t)g2 * hkv_g * d * es;
        s = attention_dispatch(ctx, gs, *params, dQ + off, static_cast<char*>(dK) + kv_off, static_cast<char*>(dV) + kv_off, dI, dN,
                               dO + off, kv_compact, st);
        if (s != TF_OK) break;
        e = cudaEventRecord(ev_att, st);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(ctx->s_out, ev_att, 0);
        if (e == cudaSuccess)
            e = cudaMemcpy2DAsync(static_cast<char*>(O_host) + off, row, dO + off, row, row_g, tokens, cudaMemcpyDeviceToHost, ctx->s_out);
        if (e != cudaSuccess) s = TF_ERR_CUDA;
    }
    ctx->workspace = saved_ws; ctx->workspace_bytes = saved_bytes;
    if (s == TF_OK) {
        e = cudaStreamWaitEvent(ctx->s_out, ev_sel, 0);
        if (e == cudaSuccess && score_host) e = cudaMemcpyAsync(score_host, dS, tokens * 4, cudaMemcpyDeviceToHost, ctx->s_out);
        if (e == cudaSuccess && keep_mask_host) e = cudaMemcpyAsync(keep_mask_host, dM, tokens, cudaMemcpyDeviceToHost, ctx->s_out);
        if (e == cudaSuccess && kept_idx_host) e = cudaMemcpyAsync(kept_idx_host, dI, tokens * 4, cudaMemcpyDeviceToHost, ctx->s_out);
        if (e == cudaSuccess && n_kept_host) e = cudaMemcpyAsync(n_kept_host, dN, (size_t)shape->batch * 4, cudaMemcpyDeviceToHost, ctx->s_out);
        if (e != cudaSuccess) s = TF_ERR_CUDA;
    }
    // results are in host memory when the call returns (also drains the internal streams after an error)
    const cudaError_t e1 = cudaStreamSynchronize(ctx->s_in), e2 = cudaStreamSynchronize(st), e3 = cudaStreamSynchronize(ctx->s_out);
    if (s == TF_OK && (e1 != cudaSuccess || e2 != cudaSuccess || e3 != cudaSuccess)) s = TF_ERR_CUDA;
    return s;
}

tf_status tf_decode_step(tf_ctx* ctx, const tf_shape* shape, const tf_filter_params* params, float eta,
                         int32_t alg1_sign, const void* q_new, const void* K_cache, const void* V_cache,
                         const int32_t* pos, const tf_decode_state* state, void* O_new, float* score,
                         uint8_t* skip, void* stream) {
    if (!ctx) return TF_ERR_INVALID_ARG;
    tf_status s = check_shape(shape);
    if (s == TF_OK) s = check_params(params);
    if (s == TF_OK) s = check_kv(shape, K_cache, V_cache);
    if (s != TF_OK) return s;
    if (!q_new || !O_new || !pos || !skip || !state) return TF_ERR_INVALID_ARG;
    if (!state->sum_k || !state->sum_v || !state->count || !state->tau || !state->steps || !state->skips)
        return TF_ERR_INVALID_ARG;
    if (!(eta >= 0.f)) return TF_ERR_INVALID_ARG;
    if (params->kv_visibility != TF_KV_ALL) return TF_ERR_UNSUPPORTED;
    if (shape->q_stride[2] <= 0 || shape->o_stride[2] <= 0) return TF_ERR_UNSUPPORTED;
    DeviceGuard g(ctx->device);
    if (!g.ok) return TF_ERR_CUDA;
    tf::tf_decode_args a{q_new, K_cache, V_cache, pos, state, O_new, score, skip, eta, alg1_sign ? 1 : 0};
    cudaError_t e = launch_decode_step(ctx, *shape, *params, a, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? TF_OK : TF_ERR_CUDA;
}

tf_status tf_tail_policy(double p_global, double tail_fraction, int32_t n_layers, double* ratio_per_layer,
                         int32_t* n_tail_out) {
    if (!ratio_per_layer || n_layers <= 0) return TF_ERR_INVALID_ARG;
    if (!(p_global >= 0.0 && p_global < 1.0) || !(tail_fraction > 0.0 && tail_fraction <= 1.0)) return TF_ERR_INVALID_ARG;
    const double p_tail = p_global / tail_fraction;
    if (!(p_tail < 1.0)) return TF_ERR_INVALID_ARG;
    int n_tail = (int)floor(tail_fraction * (double)n_layers + 0.5);
    if (n_tail < 1) n_tail = 1;
    if (n_tail > n_layers) n_tail = n_layers;
    for (int l = 0; l < n_layers; ++l) ratio_per_layer[l] = (l >= n_layers - n_tail) ? p_tail : 0.0;
    if (n_tail_out) *n_tail_out = n_tail;
    return TF_OK;
}

tf_status tf_get_status(tf_ctx* ctx, int sync, int64_t detail[4]) {
    if (!ctx) return TF_ERR_INVALID_ARG;
    DeviceGuard g(ctx->device);
    if (!g.ok) return TF_ERR_CUDA;
    if (sync && cudaDeviceSynchronize() != cudaSuccess) return TF_ERR_CUDA;
    DevStatus h{};
    if (cudaMemcpy(&h, ctx->dev_status, sizeof(h), cudaMemcpyDeviceToHost) != cudaSuccess) return TF_ERR_CUDA;
    if (detail) {
        detail[0] = (int64_t)h.code; detail[1] = (int64_t)h.where;
        detail[2] = (int64_t)h.nan_count; detail[3] = (int64_t)ctx->launches;
    }
    if (h.code == TF_ERR_TIMEOUT) {
        invalidate_scan_scratch(ctx);   // records written under a wait that gave up are not to be trusted
        return TF_ERR_TIMEOUT;
    }
    if (h.code == TF_ERR_NAN_SCORE) return TF_ERR_NAN_SCORE;
    return TF_OK;
}

tf_status tf_clear_status(tf_ctx* ctx) {
    if (!ctx) return TF_ERR_INVALID_ARG;
    DeviceGuard g(ctx->device);
    if (!g.ok) return TF_ERR_CUDA;
    invalidate_scan_scratch(ctx);
    return cudaMemset(ctx->dev_status, 0, sizeof(DevStatus)) == cudaSuccess ? TF_OK : TF_ERR_CUDA;
}

tf_status tf_last_kernels(tf_ctx* ctx, int32_t kernels[2]) {
    if (!ctx || !kernels) return TF_ERR_INVALID_ARG;
    kernels[0] = ctx->last_scan_kernel;
    kernels[1] = ctx->last_attention_kernel;
    return TF_OK;
}

tf_status tf_set_wait_limits(tf_ctx* ctx, int64_t max_polls, int64_t wait_cycles) {
    if (!ctx) return TF_ERR_INVALID_ARG;
    ctx->max_polls = max_polls < 0 ? -1 : max_polls;
    ctx->wait_cycles = wait_cycles < 0 ? -1 : wait_cycles;
    return TF_OK;
}

tf_status tf_set_attention_path(tf_ctx* ctx, int use_tensor_cores) {
    if (!ctx) return TF_ERR_INVALID_ARG;
    if (use_tensor_cores < 0 || use_tensor_cores > 6) return TF_ERR_INVALID_ARG;
    ctx->use_tensor_cores = use_tensor_cores ? 1 : 0;
    ctx->attention_form = use_tensor_cores >= 2 ? use_tensor_cores - 1 : 0;
    return TF_OK;
}

tf_status tf_set_select_path(tf_ctx* ctx, int path) {
    if (!ctx || path < 0 || path > 2) return TF_ERR_INVALID_ARG;
    ctx->select_form = path;
    return TF_OK;
}

tf_status tf_set_scan_path(tf_ctx* ctx, int path) {
    if (!ctx || path < 0 || path > 3) return TF_ERR_INVALID_ARG;
    ctx->scan_path = path;
    return TF_OK;
}

const char* tf_status_string(tf_status s) {
    switch (s) {
        case TF_OK: return "ok";
        case TF_ERR_INVALID_ARG: return "invalid argument";
        case TF_ERR_UNSUPPORTED: return "unsupported shape, dtype or layout";
        case TF_ERR_WORKSPACE: return "workspace missing or too small";
        case TF_ERR_CUDA: return "CUDA call failed";
        case TF_ERR_TIMEOUT: return "a bounded device-side wait gave up";
        case TF_ERR_NAN_SCORE: return "NaN score seen";
        default: return "unknown status";
    }
}

}  // extern "C"
