// Placeholder until the tcgen05 kernel lands: bf16 attention falls through to the CUDA-core kernel.
#include "tf_common.cuh"
namespace tf {
cudaError_t launch_attention_tc(tf_ctx*, const tf_shape&, const tf_filter_params&, const void*,
                                const void*, const void*, const int32_t*, const int32_t*, void*,
                                cudaStream_t) {
    return cudaErrorNotSupported;
}
}  // namespace tf
