// Shared device helpers for the SemantiCache kernels (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "semanticache.h"

namespace sc {

constexpr int kWarp = 32;
constexpr unsigned kFull = 0xffffffffu;

// First error wins; the word may live in device or pinned host memory.
__device__ __forceinline__ void set_status(int32_t* status, int32_t code) {
    if (status != nullptr) atomicCAS(status, 0, code);
}

template <typename T> struct Elem;
template <> struct Elem<__nv_bfloat16> {
    static __device__ __forceinline__ float load(const __nv_bfloat16* p) { return __bfloat162float(*p); }
    static __device__ __forceinline__ void store(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }
};
template <> struct Elem<float> {
    static __device__ __forceinline__ float load(const float* p) { return *p; }
    static __device__ __forceinline__ void store(float* p, float v) { *p = v; }
};

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFull, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(kFull, v, o));
    return v;
}
__device__ __forceinline__ int warp_sum_i(int v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFull, v, o);
    return v;
}
__device__ __forceinline__ int warp_max_i(int v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = max(v, __shfl_xor_sync(kFull, v, o));
    return v;
}

// Inclusive scans over one warp.
__device__ __forceinline__ int warp_scan_add(int v, int lane) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int t = __shfl_up_sync(kFull, v, o);
        if (lane >= o) v += t;
    }
    return v;
}
__device__ __forceinline__ int warp_scan_max(int v, int lane) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int t = __shfl_up_sync(kFull, v, o);
        if (lane >= o) v = max(v, t);
    }
    return v;
}

inline int div_up(int64_t a, int64_t b) { return (int)((a + b - 1) / b); }

// Statistics only: kernels launched (or captured into a graph) by this library since load.
void note_launches(int n);

// --- launch entry points implemented in the .cu files (host side) ---------------------------

struct ChunkArgs {
    const int32_t* token_ids; int32_t B, n;
    int32_t delim[SC_MAX_DELIMS]; int32_t n_delim; int32_t max_chunk_len;
    int32_t* seg_off; int32_t n_seg_cap; int32_t* seq_seg_off; int32_t* n_seg;
    int32_t* tile_seg; int32_t n_tile_cap; int32_t* seq_tile_cnt;
    int32_t* ws; int32_t* status;
};
cudaError_t launch_chunk(const ChunkArgs& a, cudaStream_t st);
size_t chunk_ws_bytes(int32_t B, int32_t n);

struct CompressArgs {
    const void* K; const void* V; sc_strides st; sc_dtype dt;
    int32_t B, Hkv, n, d;
    const int32_t* seg_off; const int32_t* seq_seg_off; const int32_t* n_seg;
    const int32_t* tile_seg; const int32_t* seq_tile_cnt; int32_t n_tile_cap;
    float tau; int32_t max_chunk_len; uint32_t flags;
    void* core_k; void* core_v; int32_t* count; int32_t cap; int32_t* core_len;
    int32_t* assign; void* ws; int32_t* status;
    // budget search (all null / 0 for an ordinary call): the threshold is read from device memory; a pass
    // may be told to do nothing by a device flag; a counting pass only adds each head's cluster count to
    // core_len (which the caller zeroed) and writes nothing else
    const float* tau_dev; const int32_t* skip; int32_t count_only;
};
cudaError_t launch_compress_generic(const CompressArgs& a, cudaStream_t st);
cudaError_t launch_compress_fused_layers(const CompressArgs& a, const sc_compress_layer* layers, int32_t L, cudaStream_t st);
size_t compress_fused_layers_ws_bytes(int32_t L, int32_t B, int32_t Hkv, int32_t n);
size_t compress_generic_ws_bytes(int32_t B, int32_t Hkv, int32_t n);

struct GlobalArgs {   // clustering of whole sequences (no chunking)
    const void* K; const void* V; sc_strides st; sc_dtype dt; int32_t B, Hkv, n, d;
    float tau; uint32_t flags;
    void* core_k; void* core_v; int32_t* count; int32_t cap; int32_t* core_len; int32_t* assign;
    void* ws; int32_t* status;
};
cudaError_t launch_compress_global(const GlobalArgs& a, cudaStream_t st);
size_t compress_global_ws_bytes(int32_t B, int32_t Hkv, int32_t n);

struct DecodeArgs {
    const void* q; sc_dtype dt; int32_t B, Hq, Hkv, d;
    const void* core_k; const void* core_v; const int32_t* count; int32_t cap;
    const int32_t* core_len; float scale; uint32_t flags; void* out; void* ws; int32_t* status;
};
cudaError_t launch_decode_generic(const DecodeArgs& a, cudaStream_t st);
size_t decode_generic_ws_bytes(int32_t B, int32_t Hq, int32_t Hkv, int32_t d, int32_t cap);

struct PrefillArgs {   // Eq. 4 with a block of m queries per head
    const void* q; sc_dtype dt; int32_t B, Hq, Hkv, m, d;
    const void* core_k; const void* core_v; const int32_t* count; int32_t cap;
    const int32_t* core_len; float scale; uint32_t flags; void* out; int32_t* status;
};
cudaError_t launch_prefill(const PrefillArgs& a, cudaStream_t st);

struct AppendArgs {
    const void* k_new; const void* v_new; sc_dtype dt; int32_t B, Hkv, d;
    const int32_t* token_ids; int32_t delim[SC_MAX_DELIMS]; int32_t n_delim; int32_t max_chunk_len; float tau;
    void* core_k; void* core_v; int32_t* count; int32_t cap;
    int32_t* core_len; int32_t* tail_len; int32_t* attn_len; int32_t* status;
};
cudaError_t launch_append(const AppendArgs& a, cudaStream_t st);
cudaError_t launch_append_layers(const AppendArgs& a, const sc_append_layer* table, int32_t L, cudaStream_t st);

}  // namespace sc
