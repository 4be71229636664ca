// sc_decode_attn_static: the decode step for callers that cannot hand the library a workspace.
//
// sc_decode_attn keeps its split partials and arrival counters in scratch memory the caller
// allocates.  Some callers have no way to allocate device memory when they reach the decode loop:
// an inference server that gave every free byte of HBM to its KV-cache pool at start-up (a later
// cudaMalloc simply fails), a plug-in running inside a host runtime that forbids allocation in
// its step callback, or a latency-critical loop that cannot afford the device-wide
// synchronisation an allocation may imply.  For them the same kernels run here with the scratch
// in a fixed array that is part of the library image: SC_STATIC_SCRATCH_BYTES on every GPU that
// loads the library, held until the process exits.  Nothing in this file allocates.
#include <mutex>

#include "common.cuh"

// The scratch itself.  In host code this name is only a handle for the runtime's symbol table,
// never an address a kernel may be given; the device address is looked up per GPU below.
static __device__ __align__(256) unsigned char g_static_scratch[SC_STATIC_SCRATCH_BYTES];

namespace {

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
void* g_scratch_ptr[kMaxDevices] = {nullptr};

// Device address of g_static_scratch on the current GPU; looked up once per GPU (first call).
cudaError_t static_scratch(void** out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (g_scratch_ptr[dev] == nullptr) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess) return e;
        if (p == nullptr || (reinterpret_cast<uintptr_t>(p) & 255u) != 0) return cudaErrorInvalidSymbol;
        g_scratch_ptr[dev] = p;
    }
    *out = g_scratch_ptr[dev];
    return cudaSuccess;
}

}  // namespace

namespace sc {
bool decode_mma_supported(const DecodeArgs& a);
size_t decode_mma_counter_bytes(int32_t B, int32_t Hkv);
}  // namespace sc

extern "C" sc_status sc_decode_attn_static(const void* q, sc_dtype dt, int32_t B, int32_t Hq, int32_t Hkv,
                                           int32_t d, const void* core_k, const void* core_v,
                                           const int32_t* count, int32_t cap, const int32_t* core_len,
                                           float scale, uint32_t flags, void* out, int32_t* status,
                                           void* stream) {
    // The same checks, in the same order, as sc_decode_attn makes before it looks at its workspace.
    if (B < 0 || Hq <= 0 || Hkv <= 0 || cap < 0 || (Hq % Hkv) != 0) return SC_ERR_INVALID_ARG;
    if (dt != SC_BF16 && dt != SC_F32) return SC_ERR_UNSUPPORTED;
    if (d < 8 || d > 256 || (d % 8) != 0) return SC_ERR_UNSUPPORTED;
    if (!(scale == scale) || scale < 0.f) return SC_ERR_INVALID_ARG;
    // An overlapped launch would run beside its neighbour's clearing of the one shared array.
    if (flags & (SC_FLAG_OVERLAP_PREV | SC_FLAG_OVERLAP_CHAIN)) return SC_ERR_INVALID_ARG;
    if (B == 0) return SC_OK;
    const size_t need = sc_decode_workspace_bytes(B, Hq, Hkv, d, cap);
    if (need > (size_t)SC_STATIC_SCRATCH_BYTES) return SC_ERR_CAPACITY;   // problem too large for the fixed array
    void* scratch = nullptr;
    if (static_scratch(&scratch) != cudaSuccess) return SC_ERR_CUDA;
    // The array still holds whatever the previous call (or an aborted one) left.  Only the arrival
    // counters at its front must start at zero (the tensor-core kernel's; the generic kernels keep
    // none): every split partial is written by its block before the merging block reads it.  They
    // are cleared here, in stream order, before the kernel runs.
    sc::DecodeArgs probe = {};
    probe.dt = dt; probe.B = B; probe.Hq = Hq; probe.Hkv = Hkv; probe.d = d; probe.cap = cap;
    if (!(flags & SC_FLAG_GENERIC) && sc::decode_mma_supported(probe)) {
        if (cudaMemsetAsync(scratch, 0, sc::decode_mma_counter_bytes(B, Hkv), (cudaStream_t)stream) != cudaSuccess)
            return SC_ERR_CUDA;
    }
    return sc_decode_attn(q, dt, B, Hq, Hkv, d, core_k, core_v, count, cap, core_len, scale, flags, out, scratch,
                          (size_t)SC_STATIC_SCRATCH_BYTES, status, stream);
}
