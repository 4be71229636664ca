// Tensor-core bf16 decode path (placeholder until the kernel lands).
#include "common.cuh"
namespace sc {
bool decode_mma_supported(const DecodeArgs&) { return false; }
cudaError_t launch_decode_mma(const DecodeArgs&, cudaStream_t) { return cudaErrorNotSupported; }
size_t decode_mma_ws_bytes(int32_t, int32_t, int32_t, int32_t, int32_t) { return 0; }
}  // namespace sc
