/*
 * tf.h -- C boundary of the B200 (sm_100a) Token Filtering layer step.
 *
 * One attention layer of a prefill sequence, as the paper's Algorithm 1 defines it
 * for "the current token", applied to every token t with tokens 0..t-1 as its past:
 *
 *   tf_kv_stats          anchors (running mean of past K / V per head) and the per-head
 *                        cosine similarity of each token's K and V to them
 *   tf_score_fuse        mean / variance over heads, variance-aware weight (Eq. 2) and
 *                        fused score S_KV (Eq. 3), one per token
 *   tf_select            which tokens skip attention at the target pruning ratio (or
 *                        above a threshold, Alg. 1 "skip if s_KV > tau"), compacted
 *   tf_pruned_attention  causal attention for retained tokens only; skipped tokens'
 *                        output rows are zero (Section 3.2)
 *   tf_layer_filter      the four steps chained on one stream
 *
 * Conventions, unless an argument says otherwise:
 *   - every tensor pointer is DEVICE memory owned by the caller; the library reads its
 *     inputs, writes its outputs, keeps no pointer after the call returns;
 *   - calls enqueue work on the given CUDA stream (a cudaStream_t passed as void*,
 *     NULL = default stream), do not synchronise and do not allocate; after one call of the
 *     same shape outside a capture (it clears the scratch and sets function attributes) a call
 *     may be captured into a CUDA graph and replayed: nothing about a launch lives on the host;
 *   - the return value reports host-side validation and launch errors only; conditions
 *     found on the device (a bounded wait that gave up) are read with tf_get_status;
 *   - head_dim must be 128; Q/K/V/O rows (head_dim elements) are contiguous and 16-byte
 *     aligned, every stride a multiple of 8 elements (bf16) / 4 elements (fp32).
 */
#ifndef TF_H_
#define TF_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct tf_ctx tf_ctx; /* opaque: device id, device status word, workspace binding */

typedef enum {
    TF_OK = 0,
    TF_ERR_INVALID_ARG = 1, /* NULL required pointer, bad enum, ratio outside [0,1), ... */
    TF_ERR_UNSUPPORTED = 2, /* head_dim != 128, dtype unknown, misaligned stride          */
    TF_ERR_WORKSPACE = 3,   /* no workspace bound, or too small for this shape            */
    TF_ERR_CUDA = 4,        /* a CUDA runtime / driver call failed                        */
    TF_ERR_TIMEOUT = 5,     /* device: a bounded wait inside a kernel gave up             */
    TF_ERR_NAN_SCORE = 6    /* device: a NaN score was seen (it is never pruned)          */
} tf_status;

typedef enum { TF_F32 = 0, TF_BF16 = 1 } tf_dtype;

/* anchor_mode: what "mean of previous keys" (Section 3.2 / Alg. 1) covers */
enum { TF_ANCHOR_PAST_MEAN = 0, /* tokens strictly before t (default)                     */
       TF_ANCHOR_INCL_MEAN = 1, /* tokens up to and including t (Alg. 1 read literally)   */
       TF_ANCHOR_EMA = 2 };     /* Eq. 1: anchor <- gamma*anchor + (1-gamma)*x, compare first */
/* fuse_mode: the weight alpha of Eq. 2-3 */
enum { TF_FUSE_INVVAR = 0,      /* alpha = var_v/(var_k+var_v): lower variance weighs more */
       TF_FUSE_EQ2_LITERAL = 1, /* alpha = var_k/(var_k+var_v): Eq. 2 exactly as printed   */
       TF_FUSE_KEY_ONLY = 2, TF_FUSE_VALUE_ONLY = 3, /* criterion ablation (Section 4.3)   */
       TF_FUSE_MEAN = 4 };      /* alpha = 1/2 (Figure 1 caption)                          */
enum { TF_SELECT_RATIO = 0,     /* prune exactly P = min(E, floor(ratio*S)) top-scoring eligible tokens */
       TF_SELECT_THRESHOLD = 1 }; /* prune eligible tokens with score > threshold (strict) */
enum { TF_KV_ALL = 0,           /* retained queries see every earlier token's K/V (default) */
       TF_KV_RETAINED = 1 };    /* retained queries see retained tokens' K/V only           */

/* Problem shape.  Tensors are addressed as base + b*stride[0] + t*stride[1] + h*stride[2] + i,
 * in ELEMENTS, i in [0, head_dim).  Query head q reads KV head q / (n_q_heads / n_kv_heads). */
typedef struct {
    int32_t batch, seq, n_q_heads, n_kv_heads, head_dim;
    int32_t dtype;          /* tf_dtype of Q, K, V and O                                     */
    int64_t q_stride[3], k_stride[3], v_stride[3], o_stride[3];
    int32_t window;         /* 0: key j visible to query t iff j <= t; W>0: also j > t - W   */
    float softmax_scale;    /* 0 => 1/sqrt(head_dim)                                         */
} tf_shape;

/* Method parameters (Alg. 1 inputs and the readings of it that are selectable). */
typedef struct {
    double prune_ratio;       /* RATIO mode: target fraction of the S tokens to prune, in [0,1) */
    int32_t warmup_tokens;    /* the first n tokens of each sequence are never pruned (Section 3.2 warm-up) */
    const uint8_t *eligible;  /* optional device [B,S]: 1 = may be pruned; NULL = all             */
    int32_t anchor_mode;      /* TF_ANCHOR_*                                                      */
    float gamma;              /* EMA smoothing factor of Eq. 1 (EMA mode only)                    */
    int32_t fuse_mode;        /* TF_FUSE_*                                                        */
    float var_eps;            /* added to each variance so alpha is defined when both are 0; 0 => 1e-8 */
    int32_t select_mode;      /* TF_SELECT_*                                                      */
    const float *threshold;   /* THRESHOLD mode: device [B]                                       */
    int32_t kv_visibility;    /* TF_KV_*                                                          */
} tf_filter_params;

/* Optional anchor state carried between calls (chunked prefill, prefill -> decode): the sums
 * (EMA mode: the anchors) over all tokens seen so far, fp32 [B, n_kv_heads, head_dim], and the
 * token count per sequence [B].  Any pointer may be NULL (in: no past; out: not wanted). */
typedef struct {
    const float *sum_k_in, *sum_v_in;
    const int64_t *count_in;
    float *sum_k_out, *sum_v_out;
} tf_carry;

/* Fill p with the defaults: ratio 0.5, warm-up 1 token, past-mean anchors, inverse-variance
 * fusion, ratio selection, all K/V visible. */
void tf_default_params(tf_filter_params *p);

/* Create / destroy a context on CUDA device `device` (allocates a few words of device memory
 * for the status record; the only allocation the library makes besides tf_layer_filter_host). */
tf_status tf_create(tf_ctx **out, int device);
tf_status tf_destroy(tf_ctx *ctx);

/* Scratch the kernels need for this shape (scan look-back records, and the intermediates of
 * tf_layer_filter that the caller does not ask for).  The caller allocates it (256-byte aligned
 * device memory) and binds it; one workspace serves one call at a time. */
tf_status tf_workspace_bytes(const tf_shape *shape, const tf_filter_params *params, size_t *bytes);
tf_status tf_set_workspace(tf_ctx *ctx, void *device_ptr, size_t bytes);

/* Steps a1+a2 (Alg. 1 lines AnchorK/AnchorV and cosine_sim; Section 3.2).  Reads K and V
 * [B,S,n_kv_heads,128] once; writes sim_k, sim_v: contiguous fp32 [B,S,n_kv_heads], the cosine
 * of token t's key / value to the anchor of its past (0 where there is no past; each norm is
 * clamped at 1e-8).  carry may be NULL.  Needs the bound workspace. */
tf_status tf_kv_stats(tf_ctx *ctx, const tf_shape *shape, const tf_filter_params *params,
                      const void *K, const void *V, float *sim_k, float *sim_v,
                      const tf_carry *carry, void *stream);

/* tf_kv_stats without any allocation on anybody's part.  (The paper has no counterpart to
 * this entry; it exists for deployment only.)  Same inputs, outputs and arithmetic as
 * tf_kv_stats, but the look-back records live in a fixed array of TF_STATIC_SCRATCH_BYTES that
 * is built into the library, so no workspace has to be bound and no context is needed.  It is
 * meant for callers that cannot obtain device memory at the point of the call: a server that
 * has already given all free HBM to its KV-cache pool, code that must leave the device heap to
 * a framework's caching allocator, or a latency-critical loop that cannot afford the
 * device-wide stall of cudaMalloc / cudaFree.  The entry calls no cudaMalloc, cudaFree or
 * other allocating routine.
 *   - Runs on the CURRENT device.  ctx may be NULL; if given it must belong to the current
 *     device, and device-side conditions (a wait that gave up) are recorded in it.  With NULL
 *     they are not recorded anywhere.
 *   - Limit: shapes whose records need more than TF_STATIC_SCRATCH_BYTES return
 *     TF_ERR_WORKSPACE and launch nothing.  The need is that of the largest record layout any
 *     scan kernel may use for the shape: 2 KiB per (64 tokens (bf16) or 32 tokens (fp32),
 *     sequence, KV head) plus one eighth of that; 8 MiB covers, for example, batch 1 x 2048
 *     tokens x 32 KV heads in bf16 three times over.
 *   - The first call on each device looks up the array's device address and zeroes the part
 *     it uses; make that first call outside any stream capture.
 *   - Every GPU on which the library is loaded holds the array until the process exits.
 *   - All calls in the process share the array of their device, and it keeps what the last
 *     call left (stale records are recognised by their launch tag; the region is zeroed again
 *     when the shape's record layout changes).  Two calls whose kernels overlap on the GPU
 *     (different streams, no ordering between them) race on it: order them. */
#define TF_STATIC_SCRATCH_BYTES (8u << 20)
tf_status tf_kv_stats_static(tf_ctx *ctx, const tf_shape *shape, const tf_filter_params *params,
                             const void *K, const void *V, float *sim_k, float *sim_v,
                             const tf_carry *carry, void *stream);

/* Step a3 (Alg. 1 lines (s_k, sigma_k^2), alpha, s_KV; Eq. 2-3).  sim_k, sim_v fp32
 * [B,S,n_kv_heads] -> score fp32 [B,S].  Population variance over the KV heads. */
tf_status tf_score_fuse(tf_ctx *ctx, const tf_shape *shape, const tf_filter_params *params,
                        const float *sim_k, const float *sim_v, float *score, void *stream);

/* Step a4 (Alg. 1 "skip if s_KV > tau"; Section 3.3 target skip ratio; Section 3.2 warm-up).
 * score fp32 [B,S] -> keep_mask u8 [B,S] (1 = retained), kept_idx i32 [B,S] (ascending retained
 * positions, then -1), n_kept i32 [B], theta fp32 [B] (lowest pruned score, +inf if none;
 * may be NULL).  RATIO mode prunes the P highest-scoring eligible tokens, equal scores resolved
 * toward the later token; a NaN score is never pruned. */
tf_status tf_select(tf_ctx *ctx, const tf_shape *shape, const tf_filter_params *params,
                    const float *score, uint8_t *keep_mask, int32_t *kept_idx, int32_t *n_kept,
                    float *theta, void *stream);

/* Steps a3 + a4 in one call (Alg. 1 from "(s_k, sigma_k^2)" to the skip decision; Eq. 2-3, Section 3.3): the
 * arguments of tf_score_fuse followed by the outputs of tf_select, with the same meaning, layout and results (the
 * scores have the bits tf_score_fuse gives, the selection the outputs tf_select gives on them).  For sequences of
 * 1025 to 32768 tokens with up to 8 KV heads both steps run in one launch, a thread-block cluster per sequence;
 * otherwise as two kernels.  theta may be NULL. */
tf_status tf_score_select(tf_ctx *ctx, const tf_shape *shape, const tf_filter_params *params,
                          const float *sim_k, const float *sim_v, float *score, uint8_t *keep_mask,
                          int32_t *kept_idx, int32_t *n_kept, float *theta, void *stream);

/* Step a5 (Section 3.2: skipped tokens' attention output is zero; standard causal softmax
 * attention otherwise).  For every retained token kept_idx[b, i], i < n_kept[b], and query head
 * q: O = softmax(scale * Q.K^T over visible keys) V.  Every other row of O is set to zero, so O
 * is fully written.  kept_idx / n_kept are device arrays as tf_select writes them. */
tf_status tf_pruned_attention(tf_ctx *ctx, const tf_shape *shape, const tf_filter_params *params,
                              const void *Q, const void *K, const void *V,
                              const int32_t *kept_idx, const int32_t *n_kept, void *O, void *stream);

/* All of Algorithm 1 for one layer plus the attention it gates: kv_stats -> score_fuse ->
 * select -> pruned_attention on one stream.  score, keep_mask, kept_idx, n_kept are optional
 * outputs (NULL: kept in the workspace).  Needs the bound workspace. */
tf_status tf_layer_filter(tf_ctx *ctx, const tf_shape *shape, const tf_filter_params *params,
                          const void *Q, const void *K, const void *V, void *O,
                          float *score, uint8_t *keep_mask, int32_t *kept_idx, int32_t *n_kept,
                          void *stream);

/* The same layer step for callers whose tensors live in HOST memory (pinned memory makes the
 * copies asynchronous): copies Q, K, V to device staging buffers that the context owns and grows
 * on demand (this entry point allocates; it also binds its own workspace, and on first use creates two
 * internal streams), runs the steps of tf_layer_filter, copies O and the optional outputs back and
 * synchronises before returning.  The copies are pipelined over both directions of the host link:
 * K and V go first (steps a1-a4 need no Q), then Q arrives in up to eight groups of query heads
 * (whole KV-head groups, at least 2 MB each) while the attention of the group before runs on the
 * caller's stream and its output rows travel back.
 * shape strides describe the host tensors; they must be dense token-major [B,S,H,128]. */
tf_status tf_layer_filter_host(tf_ctx *ctx, const tf_shape *shape, const tf_filter_params *params,
                               const void *Q_host, const void *K_host, const void *V_host,
                               void *O_host, float *score_host, uint8_t *keep_mask_host,
                               int32_t *kept_idx_host, int32_t *n_kept_host, void *stream);

/* State of the online decode step, per sequence, all DEVICE memory owned by the caller:
 * sum_k, sum_v fp32 [B, n_kv_heads, 128]: sums of the keys / values seen so far (EMA mode: the anchors
 * of Eq. 1); count [B]: tokens in them; tau fp32 [B]: the layer's skip threshold; steps, skips [B]:
 * decisions made and skips decided so far (their ratio is the running skip ratio).  sum_k, sum_v and
 * count have the layout of tf_carry, so a prefill's tf_kv_stats can fill them (sum_*_out, count = S). */
typedef struct {
    float *sum_k, *sum_v;
    int64_t *count;
    float *tau;
    int64_t *steps, *skips;
} tf_decode_state;

/* One decoding iteration of one layer (Algorithm 1 as printed, one new token per sequence): cosine of
 * the current token's key / value to the anchors in `state`, (mean, var) over heads, alpha, s_KV;
 * threshold adaptation tau += eta * (skip ratio so far - params->prune_ratio)   (Section 3.3,
 * "T_l <- T_l + eta (P_current - P_tail)"; alg1_sign != 0 uses Algorithm 1's printed sign instead);
 * the token skips attention iff s_KV > tau and pos >= params->warmup_tokens (decisions inside the
 * warm-up still count toward the ratio); the anchors take the token in; unless skipped, the token's
 * attention output is computed against cache positions <= pos (shape->window applies), else it is 0.
 *   shape: batch, n_q_heads, n_kv_heads, dtype; seq = capacity of the caches; k_stride / v_stride
 *          address K_cache / V_cache [B, seq, n_kv_heads, 128]; q_stride[0], q_stride[2] are the batch
 *          and head strides of q_new [B, n_q_heads, 128], o_stride[0], o_stride[2] those of O_new.
 *   pos:   device int32 [B], 0 <= pos[b] < seq, the cache row that already holds the current token.
 *   score (may be NULL) fp32 [B]; skip u8 [B] (required): 1 = attention skipped, O_new row is zero.
 * Two or three launches on the stream; the state is advanced in place.  If a workspace is bound
 * (tf_set_workspace, any size tf_workspace_bytes returns for a prefill of this shape is enough: the
 * need is batch * n_q_heads * splits * 520 bytes), bf16 calls split the visible keys over several CTAs
 * per KV head and keep their partial results there; without one each KV head is one CTA. */
tf_status tf_decode_step(tf_ctx *ctx, const tf_shape *shape, const tf_filter_params *params,
                         float eta, int32_t alg1_sign, const void *q_new, const void *K_cache,
                         const void *V_cache, const int32_t *pos, const tf_decode_state *state,
                         void *O_new, float *score, uint8_t *skip, void *stream);

/* Tail-focused layer policy (Section 3.3, "P_tail = P_global / Y").  Host-only helper: fills
 * ratio_per_layer[0 .. n_layers) (HOST memory) with the pruning ratio each layer should be run
 * at so that the whole stack meets the global budget: the last n_tail = round(tail_fraction *
 * n_layers) layers (at least one) get p_global / tail_fraction, all earlier layers get 0 (they
 * are not filtered at all, so they pay no scoring overhead).  n_tail_out (may be NULL) receives
 * n_tail.  TF_ERR_INVALID_ARG if a ratio is outside [0,1), tail_fraction outside (0,1], or the
 * per-layer ratio would reach 1. */
tf_status tf_tail_policy(double p_global, double tail_fraction, int32_t n_layers,
                         double *ratio_per_layer, int32_t *n_tail_out);

/* Device-side conditions since the last tf_clear_status: returns TF_OK, TF_ERR_TIMEOUT or
 * TF_ERR_NAN_SCORE.  sync != 0 synchronises the device first.  detail (may be NULL) receives
 * four words: {code, where, count of NaN scores, kernels launched by this context}.  After a
 * TF_ERR_TIMEOUT the outputs of the call that saw it are undefined; the context stays usable
 * (the next similarity scan clears its scratch records first). */
tf_status tf_get_status(tf_ctx *ctx, int sync, int64_t detail[4]);
tf_status tf_clear_status(tf_ctx *ctx);

/* Which kernel ran.  kernels[0] = the kernel of the latest similarity scan (steps a1+a2) launched
 * through this context, kernels[1] = the kernel of the latest attention (step a5); TF_KERNEL_NONE
 * before the first. */
enum { TF_KERNEL_NONE = 0,
       TF_KERNEL_SCAN_PLAIN = 1,            /* CUDA-core chained scan (fp32 inputs, EMA anchors)      */
       TF_KERNEL_SCAN_GRAM_TILE = 2,        /* tcgen05 Gram-matrix scan, one tile per CTA             */
       TF_KERNEL_SCAN_GRAM_PERSISTENT = 3,  /* tcgen05 Gram-matrix scan, persistent                   */
       TF_KERNEL_ATTN_SIMT = 10,            /* CUDA-core attention (fp32)                             */
       TF_KERNEL_ATTN_TC_SHARED = 11,       /* tcgen05 attention, two Q tiles share every K/V tile    */
       TF_KERNEL_ATTN_TC_SPLIT = 12,        /* tcgen05 attention, one Q tile, K/V tiles split         */
       TF_KERNEL_ATTN_TC_SINGLE = 13,       /* tcgen05 attention, one Q tile and one softmax group, two CTAs per SM */
       TF_KERNEL_ATTN_TC_HEAD_PAIR = 14,    /* tcgen05 attention, the same 128 rows of two query heads of one KV group share every K/V tile */
       TF_KERNEL_ATTN_TC_HEAD_QUAD = 15 };  /* tcgen05 attention, the same 64 rows of four query heads of one KV group share every K/V tile */
tf_status tf_last_kernels(tf_ctx *ctx, int32_t kernels[2]);

/* Which attention kernel a bf16 call uses: 1 = tcgen05 tensor-core kernel (default; it picks between
 * its work distributions by shape and problem size; if no tensor map can describe the caller's K/V layout it
 * uses the CUDA-core kernel), 0 = the plain CUDA-core kernel that fp32 always uses, 2 = tensor-core
 * kernel, two Q tiles per CTA sharing every K/V tile, 3 = tensor-core kernel, one Q tile per CTA with its
 * K/V tiles split between the CTA's two softmax groups, 4 = tensor-core kernel, one Q tile and one softmax group
 * per CTA, two CTAs per SM, 5 = tensor-core kernel, two query heads of one KV group per CTA (the same 128 retained
 * rows of both; needs an even number of query heads per KV head), 6 = tensor-core kernel, four query heads of one KV group
 * per CTA (the same 64 retained rows of all four; needs a multiple of four query heads per KV head).  With 2 to 6 the named
 * kernel is a requirement:
 * a call it cannot take fails with TF_ERR_UNSUPPORTED instead of running another kernel.  For A/B checks. */
tf_status tf_set_attention_path(tf_ctx *ctx, int use_tensor_cores);

/* Which kernel steps a3 / a4 use (tf_select, tf_score_select, tf_layer_filter): 0 = choose (default: a cluster of
 * CTAs per sequence for 1025 to 32768 tokens, one CTA per sequence otherwise), 1 = one CTA per sequence (step a3 as
 * a launch of its own), 2 = a cluster per sequence; a call whose sequence length it cannot take (up to 1024 or more
 * than 32768 tokens) then fails with TF_ERR_UNSUPPORTED.  Same results either way.  For A/B checks. */
tf_status tf_set_select_path(tf_ctx *ctx, int path);

/* Which kernel tf_kv_stats uses: 0 = choose (default: by dtype, anchor mode and problem size), 1 = the
 * plain CUDA-core kernel (any dtype and anchor mode), 2 = the kernel that forms 128-token Gram matrices
 * on the tensor cores, one tile per CTA, 3 = the same arithmetic as a persistent kernel (one CTA per SM,
 * six tiles in flight).  2 and 3 take bf16 with running-sum anchors; other calls then fail with
 * TF_ERR_UNSUPPORTED.  For A/B checks. */
tf_status tf_set_scan_path(tf_ctx *ctx, int path);

/* Limits of the bounded waits inside the kernels (every wait on another CTA's record or on an mbarrier
 * gives up after its limit, records TF_ERR_TIMEOUT and lets the kernel finish).  max_polls: how often one
 * look-back record is re-read before giving up (0: a record that is not there at the first look counts as
 * missing); wait_cycles: SM clock cycles one mbarrier wait may take.  A negative value restores the
 * default (about a second each).  For tests of the error path and for deployments that want a tighter bound. */
tf_status tf_set_wait_limits(tf_ctx *ctx, int64_t max_polls, int64_t wait_cycles);

/* Self-test of the bounded waits (the paper has no counterpart).  Launches one small CTA that waits, with the context's
 * limits (capped at 1000 polls and 2e7 cycles), on an mbarrier nobody arrives at and on a record nobody writes, through the
 * device functions the kernels wait with.  Afterwards tf_get_status returns TF_ERR_TIMEOUT (detail[1] = 901, 902 or 903:
 * whichever wait gave up first), the context stays usable, and tf_clear_status resets it.  Harmless by construction: every
 * one of these waits ends at its limit. */
tf_status tf_wait_selftest(tf_ctx *ctx, void *stream);

const char *tf_status_string(tf_status s);

#ifdef __cplusplus
}
#endif
#endif /* TF_H_ */
