// tf_kv_stats_static: the similarity scan of tf_kv_stats for callers that must not allocate
// device memory.  The look-back records the scan needs live in a fixed array that is part of
// the library image, so the call needs neither a bound workspace nor a context.
//
// Who cannot allocate: code that runs after a serving process has handed all free HBM to its
// KV-cache pool (a cudaMalloc then fails, or steals from the pool's head room); code inside a
// framework whose caching allocator is the only party allowed to touch the device heap; and
// latency-critical loops, where the implicit device-wide synchronisation of cudaMalloc/cudaFree
// stalls every stream.  Those callers already own K, V and the two outputs; only the scratch
// was missing.
//
// Cost of the convenience: every GPU on which this library's module gets loaded carries the
// array (kStaticScratchBytes) until the process exits, whether the entry point is used or not.
//
// The array's NAME is only meaningful on the host as a handle for cudaGetSymbolAddress; it is
// not a device address.  The address is looked up once per device (with that device current),
// the return code is checked, and the looked-up pointer is what the kernel receives.
#include <mutex>

#include "tf_common.cuh"

namespace {

constexpr size_t kStaticScratchBytes = TF_STATIC_SCRATCH_BYTES;
constexpr int kMaxDevices = 64;

static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

struct DeviceSlot {
    bool ready = false;
    tf::ScanScratch scan;   // host-side bookkeeping (launch tag, ticket base) of this device's copy
};
DeviceSlot g_slots[kMaxDevices];
std::mutex g_mutex;

}  // namespace

extern "C" tf_status tf_kv_stats_static(tf_ctx* ctx, const tf_shape* shape, const tf_filter_params* params,
                                        const void* K, const void* V, float* sim_k, float* sim_v,
                                        const tf_carry* carry, void* stream) {
    using namespace tf;
    if (!shape || !params || !K || !V || !sim_k || !sim_v) return TF_ERR_INVALID_ARG;
    if (shape->batch < 0 || shape->seq < 0 || shape->n_kv_heads <= 0) return TF_ERR_INVALID_ARG;
    if (shape->head_dim != kHeadDim) return TF_ERR_UNSUPPORTED;
    if (shape->dtype != TF_F32 && shape->dtype != TF_BF16) return TF_ERR_UNSUPPORTED;
    if ((long long)shape->batch * shape->seq > (1ll << 31) - 1 || shape->batch > 65535) return TF_ERR_UNSUPPORTED;
    if (params->anchor_mode < TF_ANCHOR_PAST_MEAN || params->anchor_mode > TF_ANCHOR_EMA) return TF_ERR_INVALID_ARG;
    if (params->anchor_mode == TF_ANCHOR_EMA && !(params->gamma > 0.f && params->gamma < 1.f)) return TF_ERR_INVALID_ARG;
    const int64_t m = shape->dtype == TF_BF16 ? 8 : 4;   // strides in units of one 16-byte vector
    for (int i = 0; i < 3; ++i)
        if (shape->k_stride[i] % m || shape->v_stride[i] % m || shape->k_stride[i] < 0 || shape->v_stride[i] < 0)
            return TF_ERR_UNSUPPORTED;
    if (shape->k_stride[1] == 0 || shape->k_stride[2] == 0 || shape->v_stride[1] == 0 || shape->v_stride[2] == 0)
        return TF_ERR_UNSUPPORTED;
    if ((reinterpret_cast<uintptr_t>(K) | reinterpret_cast<uintptr_t>(V)) & 15u) return TF_ERR_UNSUPPORTED;

    // the whole point of this entry: a shape whose records do not fit is refused, never grown
    if (scan_scratch_bytes(*shape) > kStaticScratchBytes) return TF_ERR_WORKSPACE;

    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return TF_ERR_CUDA;
    if (ctx && ctx->device != dev) return TF_ERR_INVALID_ARG;

    std::lock_guard<std::mutex> lock(g_mutex);
    DeviceSlot& slot = g_slots[dev];
    if (!slot.ready) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || ptr == nullptr) {
            cudaGetLastError();
            return TF_ERR_CUDA;
        }
        slot.scan = ScanScratch();
        slot.scan.ptr = ptr;      // needs_clear is set: the first launch zeroes the record region
        slot.scan.capacity = kStaticScratchBytes;
        slot.ready = true;
    }
    tf_ctx local{};               // without a context nothing records device-side conditions
    local.device = dev;
    local.max_polls = local.wait_cycles = -1;
    tf_ctx* use = ctx ? ctx : &local;
    cudaError_t e = launch_kv_stats(use, *shape, *params, K, V, sim_k, sim_v, carry, &slot.scan,
                                    static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? TF_OK : (e == cudaErrorNotSupported ? TF_ERR_UNSUPPORTED : TF_ERR_CUDA);
}

void tf::static_scratch_invalidate(int device) {
    if (device < 0 || device >= kMaxDevices) return;
    std::lock_guard<std::mutex> lock(g_mutex);
    g_slots[device].scan.needs_clear = true;
}
