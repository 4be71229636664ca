// Fused bf16 compress path (placeholder until the tile kernel lands).
#include "common.cuh"
namespace sc {
bool compress_fused_supported(const CompressArgs&) { return false; }
cudaError_t launch_compress_fused(const CompressArgs&, cudaStream_t) { return cudaErrorNotSupported; }
size_t compress_fused_ws_bytes(int32_t, int32_t, int32_t) { return 0; }
}  // namespace sc
