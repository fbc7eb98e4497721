// tf_wait_selftest: the bounded waits of the kernels, run against conditions that never come true.
//
// Every wait inside this library's kernels (on an mbarrier, or on a tagged packet another CTA publishes) has a
// limit; when it runs out the kernel records TF_ERR_TIMEOUT and goes on.  In normal operation no wait ever runs
// out, so this entry point exists to exercise that path on purpose and harmlessly: one small CTA waits, with the
// context's limits (tf_set_wait_limits), on an mbarrier nobody arrives at and on a packet nobody writes, through
// the very device functions the kernels use.  Nothing hangs and nothing traps; the kernel ends after the limits.
#include <algorithm>

#include "tf_ptx.cuh"

namespace tf {
namespace {

__global__ void __launch_bounds__(64) wait_selftest_kernel(DevStatus* status, const uint2* never_written, unsigned int tag,
                                                            int max_polls, long long wait_cycles, unsigned int* outcome) {
    __shared__ __align__(8) unsigned long long bar_mem;
    __shared__ int abort_flag;
    const uint32_t bar = smem_u32(&bar_mem);
    if (threadIdx.x == 0) {
        mbar_init(bar, 1);
        abort_flag = 0;
        mbar_fence_init();
    }
    __syncthreads();
    unsigned int seen = 0;
    if (threadIdx.x == 0) {            // spinning wait on a barrier phase that never completes
        if (!mbar_wait_bounded(bar, 0, &abort_flag, wait_cycles, status, 901)) seen |= 1u;
    }
    __syncthreads();
    if (threadIdx.x == 0) abort_flag = 0;
    __syncthreads();
    if (threadIdx.x == 32) {           // parked wait (the form the persistent kernels use)
        if (!mbar_wait_parked(bar, 0, &abort_flag, wait_cycles, status, 902)) seen |= 2u;
    }
    if (threadIdx.x == 1) {            // a packet that never gets this launch's tag
        const uint2 first = ld_packet2(never_written);
        const float v = wait_packet2(never_written, first, tag, max_polls, status, 903);
        if (v == 0.f) seen |= 4u;
    }
    if (seen) atomicOr(outcome, seen);
}

}  // namespace
}  // namespace tf

extern "C" tf_status tf_wait_selftest(tf_ctx* ctx, void* stream) {
    using namespace tf;
    if (!ctx) return TF_ERR_INVALID_ARG;
    int prev = -1;
    if (cudaGetDevice(&prev) != cudaSuccess) return TF_ERR_CUDA;
    if (prev != ctx->device && cudaSetDevice(ctx->device) != cudaSuccess) return TF_ERR_CUDA;
    // the status record's reserved word serves as the packet nobody writes (tag 0xffffffff never occurs there) and,
    // afterwards, as the bit mask of the waits that gave up
    const uint2* never = reinterpret_cast<const uint2*>(&ctx->dev_status->reserved);
    unsigned int* outcome = reinterpret_cast<unsigned int*>(&ctx->dev_status->reserved);
    // the limits are capped here: the self-test is meant to take microseconds to milliseconds, whatever the context's limits
    const int polls = (int)std::min<long long>(ctx_max_polls(ctx), 1000);
    const long long cycles = std::min<long long>(ctx_wait_cycles(ctx), 20000000ll);
    wait_selftest_kernel<<<1, 64, 0, static_cast<cudaStream_t>(stream)>>>(ctx->dev_status, never, 0xffffffffu, polls, cycles, outcome);
    ctx->launches += 1;
    const cudaError_t e = cudaGetLastError();
    if (prev != ctx->device) cudaSetDevice(prev);
    return e == cudaSuccess ? TF_OK : TF_ERR_CUDA;
}
