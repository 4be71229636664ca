// C-ABI entry points: argument validation and dispatch.  See include/semanticache.h.
#include <math.h>

#include "common.cuh"

using namespace sc;

namespace sc {
// fused bf16 paths (compress_fused.cu, decode_mma.cu)
bool compress_fused_supported(const CompressArgs& a);
cudaError_t launch_compress_fused(const CompressArgs& a, cudaStream_t st);
size_t compress_fused_ws_bytes(int32_t B, int32_t Hkv, int32_t n);
bool decode_mma_supported(const DecodeArgs& a);
cudaError_t launch_decode_mma(const DecodeArgs& a, cudaStream_t st);
size_t decode_mma_ws_bytes(int32_t B, int32_t Hq, int32_t Hkv, int32_t d, int32_t cap);
size_t budget_state_bytes();
cudaError_t launch_compress_budget(CompressArgs a, void* ws_compress, void* ws_generic, const float* grid, int n_grid,
                                   long long target, float* tau_out, int32_t* search_out, cudaStream_t st);
}  // namespace sc

#include <atomic>
static std::atomic<uint64_t> g_launches{0};
namespace sc { void note_launches(int n) { g_launches.fetch_add((uint64_t)n, std::memory_order_relaxed); } }

static inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
static inline int tile_cap_for(int32_t n) { return 2 * div_up(n, SC_TILE_ROWS) + 1; }
static inline size_t fused_region_bytes(int32_t B, int32_t Hkv, int32_t n) {
    return (compress_fused_ws_bytes(B, Hkv, n) + 255) / 256 * 256;
}

extern "C" {

const char* sc_version(void) { return "semanticache-b200 0.1 (sm_100a)"; }

uint64_t sc_launch_counter(void) { return g_launches.load(std::memory_order_relaxed); }

sc_status sc_chunk_bounds(int32_t B, int32_t n, int32_t* n_seg_cap, int32_t* n_tile_cap) {
    if (B < 0 || n < 0 || (int64_t)B * n > 0x7fffffff - 1) return SC_ERR_INVALID_ARG;
    if (n_seg_cap) *n_seg_cap = B * n;
    if (n_tile_cap) *n_tile_cap = tile_cap_for(n);
    return SC_OK;
}

size_t sc_chunk_workspace_bytes(int32_t B, int32_t n) {
    if (B <= 0 || n <= 0) return 256;
    return chunk_ws_bytes(B, n);
}

sc_status sc_chunk(const int32_t* token_ids, int32_t B, int32_t n, const int32_t* delim_ids, int32_t n_delim,
                   int32_t max_chunk_len, int32_t* seg_off, int32_t n_seg_cap, int32_t* seq_seg_off,
                   int32_t* n_seg, int32_t* tile_seg, int32_t n_tile_cap, int32_t* seq_tile_cnt,
                   void* workspace, size_t workspace_bytes, int32_t* status, void* stream) {
    if (B < 0 || n < 0 || (int64_t)B * n > 0x7fffffff - 1) return SC_ERR_INVALID_ARG;
    if (n_delim < 0 || n_delim > SC_MAX_DELIMS || (n_delim > 0 && !delim_ids)) return SC_ERR_INVALID_ARG;
    if (max_chunk_len < 1 || max_chunk_len > SC_MAX_CHUNK_LEN) return SC_ERR_INVALID_ARG;
    if (!seg_off || !seq_seg_off || !n_seg || !tile_seg || !seq_tile_cnt) return SC_ERR_INVALID_ARG;
    if (n_seg_cap < 0 || n_tile_cap < 0) return SC_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    if (B == 0 || n == 0) {  // nothing to chunk: empty offsets
        cudaError_t e = cudaMemsetAsync(n_seg, 0, sizeof(int32_t), st);
        if (e == cudaSuccess) e = cudaMemsetAsync(seq_seg_off, 0, sizeof(int32_t) * (B + 1), st);
        if (e == cudaSuccess) e = cudaMemsetAsync(seg_off, 0, sizeof(int32_t), st);
        if (e == cudaSuccess && B > 0) e = cudaMemsetAsync(seq_tile_cnt, 0, sizeof(int32_t) * B, st);
        for (int b = 0; e == cudaSuccess && b < B; ++b)
            e = cudaMemsetAsync(tile_seg + (int64_t)b * (n_tile_cap + 1), 0, sizeof(int32_t), st);
        return e == cudaSuccess ? SC_OK : SC_ERR_CUDA;
    }
    if (!token_ids || !workspace || workspace_bytes < chunk_ws_bytes(B, n)) return SC_ERR_INVALID_ARG;
    ChunkArgs a;
    a.token_ids = token_ids; a.B = B; a.n = n;
    for (int i = 0; i < SC_MAX_DELIMS; ++i) a.delim[i] = i < n_delim ? delim_ids[i] : 0;
    a.n_delim = n_delim; a.max_chunk_len = max_chunk_len;
    a.seg_off = seg_off; a.n_seg_cap = n_seg_cap; a.seq_seg_off = seq_seg_off; a.n_seg = n_seg;
    a.tile_seg = tile_seg; a.n_tile_cap = n_tile_cap; a.seq_tile_cnt = seq_tile_cnt;
    a.ws = (int32_t*)workspace; a.status = status;
    return launch_chunk(a, st) == cudaSuccess ? SC_OK : SC_ERR_CUDA;
}

size_t sc_compress_workspace_bytes(int32_t B, int32_t Hkv, int32_t n) {
    if (B <= 0 || Hkv <= 0 || n <= 0) return 256;
    // [status words and counters of the fused kernel (zero between calls)] [scratch of the generic kernels]
    return fused_region_bytes(B, Hkv, n) + compress_generic_ws_bytes(B, Hkv, n);
}

sc_status sc_compress(const void* K, const void* V, sc_strides kv_strides, sc_dtype dt, int32_t B, int32_t Hkv,
                      int32_t n, int32_t d, const int32_t* seg_off, const int32_t* seq_seg_off,
                      const int32_t* n_seg, const int32_t* tile_seg, const int32_t* seq_tile_cnt,
                      int32_t n_tile_cap, const sc_gsc_params* params, void* core_k, void* core_v, int32_t* count,
                      int32_t cap, int32_t* core_len, int32_t* assign, void* workspace, size_t workspace_bytes,
                      int32_t* status, void* stream) {
    if (B < 0 || Hkv <= 0 || n < 0 || cap < 0 || !params || !core_len) return SC_ERR_INVALID_ARG;
    if (dt != SC_BF16 && dt != SC_F32) return SC_ERR_UNSUPPORTED;
    if (d < 8 || d > 256 || (d % 8) != 0) return SC_ERR_UNSUPPORTED;
    if (params->max_chunk_len < 1 || params->max_chunk_len > SC_MAX_CHUNK_LEN) return SC_ERR_INVALID_ARG;
    if (!(params->tau == params->tau)) return SC_ERR_INVALID_ARG;  // NaN threshold
    cudaStream_t st = (cudaStream_t)stream;
    if (B == 0 || n == 0) {
        if (B == 0) return SC_OK;
        return cudaMemsetAsync(core_len, 0, sizeof(int32_t) * (size_t)B * Hkv, st) == cudaSuccess ? SC_OK : SC_ERR_CUDA;
    }
    if (!K || !V || !seg_off || !seq_seg_off || !n_seg || !tile_seg || !seq_tile_cnt) return SC_ERR_INVALID_ARG;
    if (!core_k || !core_v || !count || !workspace) return SC_ERR_INVALID_ARG;
    if (!aligned16(K) || !aligned16(V) || !aligned16(core_k) || !aligned16(core_v)) return SC_ERR_INVALID_ARG;
    const size_t esz = dt == SC_BF16 ? 2 : 4;
    if ((kv_strides.b * esz) % 16 || (kv_strides.h * esz) % 16 || (kv_strides.n * esz) % 16) return SC_ERR_INVALID_ARG;
    if (kv_strides.n < d) return SC_ERR_INVALID_ARG;
    if ((int64_t)B * n > 0x7fffffff - 1) return SC_ERR_INVALID_ARG;
    if (n_tile_cap < 1 || n_tile_cap > tile_cap_for(n)) return SC_ERR_INVALID_ARG;
    if (workspace_bytes < sc_compress_workspace_bytes(B, Hkv, n)) return SC_ERR_INVALID_ARG;
    CompressArgs a;
    a.K = K; a.V = V; a.st = kv_strides; a.dt = dt; a.B = B; a.Hkv = Hkv; a.n = n; a.d = d;
    a.seg_off = seg_off; a.seq_seg_off = seq_seg_off; a.n_seg = n_seg;
    a.tile_seg = tile_seg; a.seq_tile_cnt = seq_tile_cnt; a.n_tile_cap = n_tile_cap;
    a.tau = params->tau; a.max_chunk_len = params->max_chunk_len; a.flags = params->flags;
    a.core_k = core_k; a.core_v = core_v; a.count = count; a.cap = cap; a.core_len = core_len;
    a.assign = assign; a.ws = workspace; a.status = status;
    a.tau_dev = nullptr; a.skip = nullptr; a.count_only = 0;
    cudaError_t e;
    e = cudaErrorNotSupported;
    if (!(a.flags & SC_FLAG_GENERIC) && compress_fused_supported(a)) e = launch_compress_fused(a, st);
    if (e == cudaErrorNotSupported) {   // forced, or a shape / layout the fused kernel does not take
        a.ws = (char*)workspace + fused_region_bytes(B, Hkv, n);   // never touches the fused kernel's words
        e = launch_compress_generic(a, st);
    }
    return e == cudaSuccess ? SC_OK : SC_ERR_CUDA;
}

size_t sc_compress_layers_workspace_bytes(int32_t L, int32_t B, int32_t Hkv, int32_t n) {
    if (L <= 0 || B <= 0 || Hkv <= 0 || n <= 0) return 256;
    // [status words and counters of the fused kernel for all layers] [scratch of the generic kernels, one layer at a time]
    return (compress_fused_layers_ws_bytes(L, B, Hkv, n) + 255) / 256 * 256 + compress_generic_ws_bytes(B, Hkv, n);
}

sc_status sc_compress_layers(const sc_compress_layer* layers, int32_t L, sc_strides kv_strides, sc_dtype dt, int32_t B,
                             int32_t Hkv, int32_t n, int32_t d, const int32_t* seg_off, const int32_t* seq_seg_off,
                             const int32_t* n_seg, const int32_t* tile_seg, const int32_t* seq_tile_cnt,
                             int32_t n_tile_cap, const sc_gsc_params* params, int32_t cap, void* workspace,
                             size_t workspace_bytes, int32_t* status, void* stream) {
    if (L < 0 || L > SC_MAX_LAYERS_PER_CALL || B <= 0 || Hkv <= 0 || n <= 0 || cap < 0 || !params) return SC_ERR_INVALID_ARG;
    if (dt != SC_BF16 && dt != SC_F32) return SC_ERR_UNSUPPORTED;
    if (d < 8 || d > 256 || (d % 8) != 0) return SC_ERR_UNSUPPORTED;
    if (params->max_chunk_len < 1 || params->max_chunk_len > SC_MAX_CHUNK_LEN) return SC_ERR_INVALID_ARG;
    if (!(params->tau == params->tau) || (params->flags & ~SC_FLAG_GENERIC)) return SC_ERR_INVALID_ARG;
    if (L == 0) return SC_OK;
    if (!layers || !seg_off || !seq_seg_off || !n_seg || !tile_seg || !seq_tile_cnt || !workspace) return SC_ERR_INVALID_ARG;
    const size_t esz = dt == SC_BF16 ? 2 : 4;
    if ((kv_strides.b * esz) % 16 || (kv_strides.h * esz) % 16 || (kv_strides.n * esz) % 16) return SC_ERR_INVALID_ARG;
    if (kv_strides.n < d || (int64_t)B * n > 0x7fffffff - 1) return SC_ERR_INVALID_ARG;
    if (n_tile_cap < 1 || n_tile_cap > tile_cap_for(n)) return SC_ERR_INVALID_ARG;
    if (workspace_bytes < sc_compress_layers_workspace_bytes(L, B, Hkv, n)) return SC_ERR_INVALID_ARG;
    for (int l = 0; l < L; ++l) {
        const sc_compress_layer& y = layers[l];
        if (!y.K || !y.V || !y.core_k || !y.core_v || !y.count || !y.core_len) return SC_ERR_INVALID_ARG;
        if (!aligned16(y.K) || !aligned16(y.V) || !aligned16(y.core_k) || !aligned16(y.core_v)) return SC_ERR_INVALID_ARG;
    }
    CompressArgs a = {};
    a.st = kv_strides; a.dt = dt; a.B = B; a.Hkv = Hkv; a.n = n; a.d = d;
    a.seg_off = seg_off; a.seq_seg_off = seq_seg_off; a.n_seg = n_seg;
    a.tile_seg = tile_seg; a.seq_tile_cnt = seq_tile_cnt; a.n_tile_cap = n_tile_cap;
    a.tau = params->tau; a.max_chunk_len = params->max_chunk_len; a.flags = params->flags;
    a.cap = cap; a.ws = workspace; a.status = status;
    cudaStream_t st = (cudaStream_t)stream;
    cudaError_t e = cudaErrorNotSupported;
    if (!(a.flags & SC_FLAG_GENERIC)) {
        CompressArgs probe = a;   // what compress_fused_supported looks at is shared by the layers
        if (compress_fused_supported(probe)) e = launch_compress_fused_layers(a, layers, L, st);
    }
    if (e == cudaErrorNotSupported) {   // forced, or a shape / layout the fused kernel does not take: layer after layer
        a.ws = (char*)workspace + (compress_fused_layers_ws_bytes(L, B, Hkv, n) + 255) / 256 * 256;
        e = cudaSuccess;
        for (int l = 0; l < L && e == cudaSuccess; ++l) {
            CompressArgs g = a;
            g.K = layers[l].K; g.V = layers[l].V; g.core_k = layers[l].core_k; g.core_v = layers[l].core_v;
            g.count = layers[l].count; g.core_len = layers[l].core_len; g.assign = layers[l].assign;
            e = launch_compress_generic(g, st);
        }
    }
    return e == cudaSuccess ? SC_OK : SC_ERR_CUDA;
}

size_t sc_compress_budget_workspace_bytes(int32_t B, int32_t Hkv, int32_t n) {
    return budget_state_bytes() + sc_compress_workspace_bytes(B, Hkv, n);
}

sc_status sc_compress_budget(const void* K, const void* V, sc_strides kv_strides, sc_dtype dt, int32_t B, int32_t Hkv,
                             int32_t n, int32_t d, const int32_t* seg_off, const int32_t* seq_seg_off,
                             const int32_t* n_seg, const int32_t* tile_seg, const int32_t* seq_tile_cnt,
                             int32_t n_tile_cap, const sc_gsc_params* params, const sc_budget* budget, void* core_k,
                             void* core_v, int32_t* count, int32_t cap, int32_t* core_len, int32_t* assign,
                             float* tau_out, int32_t* search_out, void* workspace, size_t workspace_bytes,
                             int32_t* status, void* stream) {
    if (B <= 0 || Hkv <= 0 || n <= 0 || cap < 0 || !params || !budget || !core_len) return SC_ERR_INVALID_ARG;
    if (dt != SC_BF16 && dt != SC_F32) return SC_ERR_UNSUPPORTED;
    if (d < 8 || d > 256 || (d % 8) != 0) return SC_ERR_UNSUPPORTED;
    if (params->max_chunk_len < 1 || params->max_chunk_len > SC_MAX_CHUNK_LEN) return SC_ERR_INVALID_ARG;
    if (params->flags & (SC_FLAG_TWO_PASS | SC_FLAG_OVERLAP_PREV | SC_FLAG_OVERLAP_CHAIN)) return SC_ERR_INVALID_ARG;
    if (budget->n_grid < 2 || budget->n_grid > SC_BUDGET_MAX_GRID) return SC_ERR_INVALID_ARG;
    if (!(budget->target_kept >= 0.f && budget->target_kept <= 1.f)) return SC_ERR_INVALID_ARG;
    if (!(budget->tau_lo < budget->tau_hi)) return SC_ERR_INVALID_ARG;   // also refuses NaN
    if (!K || !V || !seg_off || !seq_seg_off || !n_seg || !tile_seg || !seq_tile_cnt) return SC_ERR_INVALID_ARG;
    if (!core_k || !core_v || !count || !workspace) return SC_ERR_INVALID_ARG;
    if (!aligned16(K) || !aligned16(V) || !aligned16(core_k) || !aligned16(core_v)) return SC_ERR_INVALID_ARG;
    const size_t esz = dt == SC_BF16 ? 2 : 4;
    if ((kv_strides.b * esz) % 16 || (kv_strides.h * esz) % 16 || (kv_strides.n * esz) % 16) return SC_ERR_INVALID_ARG;
    if (kv_strides.n < d) return SC_ERR_INVALID_ARG;
    if ((int64_t)B * n > 0x7fffffff - 1) return SC_ERR_INVALID_ARG;
    if (n_tile_cap < 1 || n_tile_cap > tile_cap_for(n)) return SC_ERR_INVALID_ARG;
    if (workspace_bytes < sc_compress_budget_workspace_bytes(B, Hkv, n)) return SC_ERR_INVALID_ARG;
    // the grid of thresholds, in float32 arithmetic: tau_i = tau_lo + i * ((tau_hi - tau_lo) / (n_grid - 1))
    float grid[SC_BUDGET_MAX_GRID];
    {
        volatile float step = (budget->tau_hi - budget->tau_lo) / (float)(budget->n_grid - 1);
        for (int i = 0; i < budget->n_grid; ++i) {
            volatile float prod = (float)i * step;   // rounded on its own: no fused multiply-add
            grid[i] = budget->tau_lo + prod;
        }
    }
    // the target as a number of cores of the whole layer, rounded half up
    const long long target = (long long)floor((double)budget->target_kept * ((double)B * Hkv * n) + 0.5);
    CompressArgs a;
    a.K = K; a.V = V; a.st = kv_strides; a.dt = dt; a.B = B; a.Hkv = Hkv; a.n = n; a.d = d;
    a.seg_off = seg_off; a.seq_seg_off = seq_seg_off; a.n_seg = n_seg;
    a.tile_seg = tile_seg; a.seq_tile_cnt = seq_tile_cnt; a.n_tile_cap = n_tile_cap;
    a.tau = grid[0]; a.max_chunk_len = params->max_chunk_len; a.flags = params->flags;
    a.core_k = core_k; a.core_v = core_v; a.count = count; a.cap = cap; a.core_len = core_len;
    a.assign = assign; a.ws = workspace; a.status = status;
    a.tau_dev = nullptr; a.skip = nullptr; a.count_only = 0;
    char* wsc = (char*)workspace + budget_state_bytes();
    cudaError_t e = launch_compress_budget(a, wsc, wsc + fused_region_bytes(B, Hkv, n), grid, budget->n_grid, target,
                                           tau_out, search_out, (cudaStream_t)stream);
    return e == cudaSuccess ? SC_OK : SC_ERR_CUDA;
}

size_t sc_compress_global_workspace_bytes(int32_t B, int32_t Hkv, int32_t n) {
    if (B <= 0 || Hkv <= 0 || n <= 0) return 256;
    return compress_global_ws_bytes(B, Hkv, n);
}

sc_status sc_compress_global(const void* K, const void* V, sc_strides kv_strides, sc_dtype dt, int32_t B, int32_t Hkv,
                             int32_t n, int32_t d, float tau, uint32_t flags, void* core_k, void* core_v, int32_t* count,
                             int32_t cap, int32_t* core_len, int32_t* assign, void* workspace, size_t workspace_bytes,
                             int32_t* status, void* stream) {
    if (B < 0 || Hkv <= 0 || n < 0 || cap < 0 || !core_len) return SC_ERR_INVALID_ARG;
    if (dt != SC_BF16 && dt != SC_F32) return SC_ERR_UNSUPPORTED;
    if (d < 8 || d > 256 || (d % 8) != 0) return SC_ERR_UNSUPPORTED;
    if (!(tau == tau) || (flags & ~SC_FLAG_GENERIC)) return SC_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    if (B == 0) return SC_OK;
    if (n == 0) return cudaMemsetAsync(core_len, 0, sizeof(int32_t) * (size_t)B * Hkv, st) == cudaSuccess ? SC_OK : SC_ERR_CUDA;
    if (n > SC_GLOBAL_MAX_TOKENS || (int64_t)B * Hkv > 65535) return SC_ERR_UNSUPPORTED;
    if (!K || !V || !core_k || !core_v || !count || !workspace) return SC_ERR_INVALID_ARG;
    if (!aligned16(K) || !aligned16(V) || !aligned16(core_k) || !aligned16(core_v) || !aligned16(workspace)) return SC_ERR_INVALID_ARG;
    const size_t esz = dt == SC_BF16 ? 2 : 4;
    if ((kv_strides.b * esz) % 16 || (kv_strides.h * esz) % 16 || (kv_strides.n * esz) % 16) return SC_ERR_INVALID_ARG;
    if (kv_strides.n < d) return SC_ERR_INVALID_ARG;
    if (workspace_bytes < sc_compress_global_workspace_bytes(B, Hkv, n)) return SC_ERR_INVALID_ARG;
    GlobalArgs a;
    a.K = K; a.V = V; a.st = kv_strides; a.dt = dt; a.B = B; a.Hkv = Hkv; a.n = n; a.d = d; a.tau = tau; a.flags = flags;
    a.core_k = core_k; a.core_v = core_v; a.count = count; a.cap = cap; a.core_len = core_len; a.assign = assign;
    a.ws = workspace; a.status = status;
    return launch_compress_global(a, st) == cudaSuccess ? SC_OK : SC_ERR_CUDA;
}

size_t sc_decode_workspace_bytes(int32_t B, int32_t Hq, int32_t Hkv, int32_t d, int32_t cap) {
    if (B <= 0 || Hq <= 0 || Hkv <= 0 || d <= 0 || cap < 0) return 256;
    size_t a = decode_generic_ws_bytes(B, Hq, Hkv, d, cap), b = decode_mma_ws_bytes(B, Hq, Hkv, d, cap);
    return a > b ? a : b;
}

sc_status sc_decode_attn(const void* q, sc_dtype dt, int32_t B, int32_t Hq, int32_t Hkv, int32_t d,
                         const void* core_k, const void* core_v, const int32_t* count, int32_t cap,
                         const int32_t* core_len, float scale, uint32_t flags, void* out, void* workspace,
                         size_t workspace_bytes, int32_t* status, void* stream) {
    if (B < 0 || Hq <= 0 || Hkv <= 0 || cap < 0 || (Hq % Hkv) != 0) return SC_ERR_INVALID_ARG;
    if (dt != SC_BF16 && dt != SC_F32) return SC_ERR_UNSUPPORTED;
    if (d < 8 || d > 256 || (d % 8) != 0) return SC_ERR_UNSUPPORTED;
    if (!(scale == scale) || scale < 0.f) return SC_ERR_INVALID_ARG;
    if (B == 0) return SC_OK;
    if (!q || !out || !core_len || !workspace) return SC_ERR_INVALID_ARG;
    if (cap > 0 && (!core_k || !core_v)) return SC_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(out) || !aligned16(core_k) || !aligned16(core_v)) return SC_ERR_INVALID_ARG;
    if (workspace_bytes < sc_decode_workspace_bytes(B, Hq, Hkv, d, cap)) return SC_ERR_INVALID_ARG;
    DecodeArgs a;
    a.q = q; a.dt = dt; a.B = B; a.Hq = Hq; a.Hkv = Hkv; a.d = d; a.core_k = core_k; a.core_v = core_v;
    a.count = count; a.cap = cap; a.core_len = core_len; a.scale = scale; a.flags = flags; a.out = out; a.ws = workspace;
    a.status = status;
    cudaError_t e;
    if (!(flags & SC_FLAG_GENERIC) && decode_mma_supported(a)) e = launch_decode_mma(a, (cudaStream_t)stream);
    else e = launch_decode_generic(a, (cudaStream_t)stream);
    return e == cudaSuccess ? SC_OK : SC_ERR_CUDA;
}

sc_status sc_prefill_attn(const void* q, sc_dtype dt, int32_t B, int32_t Hq, int32_t Hkv, int32_t m, int32_t d,
                          const void* core_k, const void* core_v, const int32_t* count, int32_t cap,
                          const int32_t* core_len, float scale, uint32_t flags, void* out, int32_t* status, void* stream) {
    if (B < 0 || Hq <= 0 || Hkv <= 0 || m < 0 || cap < 0 || (Hq % Hkv) != 0) return SC_ERR_INVALID_ARG;
    if (dt != SC_BF16 && dt != SC_F32) return SC_ERR_UNSUPPORTED;
    if (d < 8 || d > 256 || (d % 8) != 0) return SC_ERR_UNSUPPORTED;
    if (!(scale == scale) || scale < 0.f || (flags & ~(SC_FLAG_GENERIC | SC_FLAG_CAUSAL_TAIL))) return SC_ERR_INVALID_ARG;
    if (B == 0 || m == 0) return SC_OK;
    if (!q || !out || !core_len) return SC_ERR_INVALID_ARG;
    if (cap > 0 && (!core_k || !core_v)) return SC_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(out) || !aligned16(core_k) || !aligned16(core_v)) return SC_ERR_INVALID_ARG;
    PrefillArgs a;
    a.q = q; a.dt = dt; a.B = B; a.Hq = Hq; a.Hkv = Hkv; a.m = m; a.d = d; a.core_k = core_k; a.core_v = core_v;
    a.count = count; a.cap = cap; a.core_len = core_len; a.scale = scale; a.flags = flags; a.out = out; a.status = status;
    return launch_prefill(a, (cudaStream_t)stream) == cudaSuccess ? SC_OK : SC_ERR_CUDA;
}

sc_status sc_append(const void* k_new, const void* v_new, sc_dtype dt, int32_t B, int32_t Hkv, int32_t d,
                    const int32_t* token_ids, const int32_t* delim_ids, int32_t n_delim, int32_t max_chunk_len,
                    float tau, void* core_k, void* core_v, int32_t* count, int32_t cap, int32_t* core_len,
                    int32_t* tail_len, int32_t* attn_len, int32_t* status, void* stream) {
    if (B < 0 || Hkv <= 0 || d <= 0 || cap < 0) return SC_ERR_INVALID_ARG;
    if (dt != SC_BF16 && dt != SC_F32) return SC_ERR_UNSUPPORTED;
    if (n_delim < 0 || n_delim > SC_MAX_DELIMS || (n_delim > 0 && !delim_ids)) return SC_ERR_INVALID_ARG;
    if (max_chunk_len < 1 || max_chunk_len > SC_MAX_CHUNK_LEN) return SC_ERR_INVALID_ARG;
    if (!(tau == tau)) return SC_ERR_INVALID_ARG;
    if (B == 0) return SC_OK;
    if (!k_new || !v_new || !token_ids || !core_k || !core_v || !count || !core_len || !tail_len || !attn_len)
        return SC_ERR_INVALID_ARG;
    AppendArgs a;
    a.k_new = k_new; a.v_new = v_new; a.dt = dt; a.B = B; a.Hkv = Hkv; a.d = d; a.token_ids = token_ids;
    for (int i = 0; i < n_delim; ++i) a.delim[i] = delim_ids[i];
    a.n_delim = n_delim; a.max_chunk_len = max_chunk_len; a.tau = tau;
    a.core_k = core_k; a.core_v = core_v; a.count = count; a.cap = cap;
    a.core_len = core_len; a.tail_len = tail_len; a.attn_len = attn_len; a.status = status;
    return launch_append(a, (cudaStream_t)stream) == cudaSuccess ? SC_OK : SC_ERR_CUDA;
}

sc_status sc_append_layers(const sc_append_layer* layers, int32_t L, sc_dtype dt, int32_t B, int32_t Hkv, int32_t d,
                           const int32_t* token_ids, const int32_t* delim_ids, int32_t n_delim, int32_t max_chunk_len,
                           float tau, int32_t cap, int32_t* status, void* stream) {
    if (B < 0 || Hkv <= 0 || d <= 0 || cap < 0 || L < 0 || L > 65535) return SC_ERR_INVALID_ARG;
    if (dt != SC_BF16 && dt != SC_F32) return SC_ERR_UNSUPPORTED;
    if (n_delim < 0 || n_delim > SC_MAX_DELIMS || (n_delim > 0 && !delim_ids)) return SC_ERR_INVALID_ARG;
    if (max_chunk_len < 1 || max_chunk_len > SC_MAX_CHUNK_LEN) return SC_ERR_INVALID_ARG;
    if (!(tau == tau)) return SC_ERR_INVALID_ARG;
    if (B == 0 || L == 0) return SC_OK;
    if (!layers || !token_ids) return SC_ERR_INVALID_ARG;
    AppendArgs a = {};
    a.dt = dt; a.B = B; a.Hkv = Hkv; a.d = d; a.token_ids = token_ids;
    for (int i = 0; i < n_delim; ++i) a.delim[i] = delim_ids[i];
    a.n_delim = n_delim; a.max_chunk_len = max_chunk_len; a.tau = tau; a.cap = cap; a.status = status;
    return launch_append_layers(a, layers, L, (cudaStream_t)stream) == cudaSuccess ? SC_OK : SC_ERR_CUDA;
}

}  // extern "C"
