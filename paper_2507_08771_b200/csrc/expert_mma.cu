// Expert stage, bulk-copy staged tensor-core variant (placeholder until it lands).
#include "common.cuh"

bool expert_mma_supported(const blockffn_ctx*, int) { return false; }
size_t expert_mma_h_bytes(const blockffn_config*) { return 256; }
cudaError_t expert_mma_setup(blockffn_ctx*) { return cudaSuccess; }
cudaError_t launch_expert_mma(blockffn_ctx*, const blockffn_weights*, const void*, const float*,
                              int, const int32_t*, const int32_t*, float*, void*, int,
                              cudaStream_t) {
  return cudaErrorNotSupported;
}
