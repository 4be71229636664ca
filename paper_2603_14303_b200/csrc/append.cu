// sc_append: one generated token joins a layer's compressed cache.
//
// The paper compresses the prompt's cache once and says nothing about the tokens generated
// afterwards.  Here they are stored behind the cores with count 1 (an "open tail" that decode
// attends to like any other row), and the chunking rule of Eq. 1 is applied on the fly: when a
// delimiter arrives, or the tail reaches max_chunk_len tokens, the tail is one finished chunk
// and is clustered (Algorithm 1 on Eq. 2) and mean-pooled (Eq. 3) in place, exactly as the same
// tokens would have been as part of a prompt.
//
// One block per (sequence, KV head).  Almost every call only stores one K row and one V row; a
// block whose chunk closes clusters at most SC_MAX_CHUNK_LEN rows that are a few KB behind the
// cores and still cached.  Any dtype, any d; CUDA cores only.
#include "common.cuh"

namespace sc {

namespace {

constexpr int kAppendThreads = 256;
constexpr int kAppendWarps = kAppendThreads / 32;
constexpr int kWords = SC_MAX_CHUNK_LEN / 32;

// The pointers of one layer, as sc_append_layers reads them from its device table.
struct LayerPtrs {
    const void* k_new; const void* v_new; void* core_k; void* core_v; int32_t* count;
    int32_t* core_len; int32_t* tail_len; int32_t* attn_len;
};

// One block = one (sequence, KV head) of one layer.  `a` carries the sizes, the delimiter set, tau and the
// token ids (its own pointers are not used), `p` the layer's buffers.
template <typename T>
__device__ __forceinline__ void append_block(const AppendArgs& a, const LayerPtrs& p) {
    __shared__ float norms[SC_MAX_CHUNK_LEN];
    __shared__ uint32_t assigned[kWords];                    // tokens of the tail that have a cluster
    __shared__ uint32_t members[SC_MAX_CHUNK_LEN][kWords];   // row c: the tokens of cluster c

    const int bh = blockIdx.x, b = bh / a.Hkv;
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const int d = a.d;
    T* ck = static_cast<T*>(p.core_k) + (int64_t)bh * a.cap * d;
    T* cv = static_cast<T*>(p.core_v) + (int64_t)bh * a.cap * d;
    int32_t* cnt = p.count + (int64_t)bh * a.cap;
    const T* kn = static_cast<const T*>(p.k_new) + (int64_t)bh * d;
    const T* vn = static_cast<const T*>(p.v_new) + (int64_t)bh * d;

    int cl = p.core_len[bh], tl = p.tail_len[bh];
    const int tok = a.token_ids[b];
    bool is_delim = false;
    for (int i = 0; i < a.n_delim; ++i) is_delim |= (a.delim[i] == tok);

    if (cl < 0 || tl < 0 || tl >= a.max_chunk_len || cl + tl >= a.cap) {   // no room (or a corrupt state): leave it as it is
        if (tid == 0) {
            set_status(a.status, (cl + tl >= a.cap && cl >= 0 && tl >= 0) ? SC_ERR_CAPACITY : SC_ERR_INVALID_ARG);
            p.attn_len[bh] = max(0, min(cl + tl, a.cap));
        }
        return;
    }

    // A token that is not a delimiter joins the tail first; a delimiter closes the tail as it is.
    if (!is_delim) {
        T* kr = ck + (int64_t)(cl + tl) * d;
        T* vr = cv + (int64_t)(cl + tl) * d;
        for (int c = tid; c < d; c += kAppendThreads) { kr[c] = kn[c]; vr[c] = vn[c]; }
        if (tid == 0) cnt[cl + tl] = 1;
        ++tl;
        __syncthreads();   // the row is read back below by other threads of this block
    }
    const bool closing = is_delim ? (tl > 0) : (tl == a.max_chunk_len);

    if (closing && tl >= 2) {
        const T* K0 = ck + (int64_t)cl * d;   // the tail: rows [0, tl)
        // ---- Eq. 2: norms ----
        for (int i = w; i < tl; i += kAppendWarps) {
            const T* row = K0 + (int64_t)i * d;
            float acc = 0.f;
            for (int c = lane; c < d; c += 32) { const float x = Elem<T>::load(row + c); acc = fmaf(x, x, acc); }
            acc = warp_sum(acc);
            if (lane == 0) norms[i] = sqrtf(acc);
        }
        if (tid < kWords) assigned[tid] = 0u;
        __syncthreads();
        // ---- Algorithm 1: the lowest token without a cluster seeds one; every later token without a
        //      cluster is compared with the seed's original key, one warp per candidate ----
        int P = 0;
        for (int i = 0; i < tl; ++i) {
            if ((assigned[i >> 5] >> (i & 31)) & 1u) continue;   // same answer in every thread: read after a barrier
            if (tid < kWords) members[P][tid] = (tid == (i >> 5)) ? (1u << (i & 31)) : 0u;
            __syncthreads();
            const T* srow = K0 + (int64_t)i * d;
            const float ni = norms[i];
            for (int j = i + 1 + w; j < tl; j += kAppendWarps) {
                if ((assigned[j >> 5] >> (j & 31)) & 1u) continue;   // bit j changes only in this warp
                const T* row = K0 + (int64_t)j * d;
                float acc = 0.f;
                for (int c = lane; c < d; c += 32) acc = fmaf(Elem<T>::load(srow + c), Elem<T>::load(row + c), acc);
                acc = warp_sum(acc);
                const float nj = norms[j];
                const float sim = (ni == 0.f || nj == 0.f) ? 0.f : acc / (ni * nj);
                if (sim > a.tau && lane == 0) {
                    atomicOr(&assigned[j >> 5], 1u << (j & 31));
                    atomicOr(&members[P][j >> 5], 1u << (j & 31));
                }
            }
            if (tid == 0) atomicOr(&assigned[i >> 5], 1u << (i & 31));
            ++P;
            __syncthreads();
        }
        // ---- Eq. 3, in place: cluster c's mean goes to tail row c.  A thread owns a column of K or of V
        //      throughout; the members of cluster c lie at rows >= c (its seed is at row >= c), and row c
        //      itself belongs to a cluster <= c, so what a thread overwrites it has already consumed ----
        for (int item = tid; item < 2 * d; item += kAppendThreads) {
            T* X = (item < d ? ck : cv) + (int64_t)cl * d + (item < d ? item : item - d);
            for (int c = 0; c < P; ++c) {
                float sum = 0.f;
                int n_mem = 0;
                for (int ww = 0; ww < kWords; ++ww) {
                    uint32_t m = members[c][ww];
                    n_mem += __popc(m);
                    while (m) {
                        const int j = ww * 32 + __ffs(m) - 1;
                        m &= m - 1;
                        sum += Elem<T>::load(X + (int64_t)j * d);
                    }
                }
                Elem<T>::store(X + (int64_t)c * d, sum / (float)n_mem);
            }
        }
        for (int c = tid; c < P; c += kAppendThreads) {
            int n_mem = 0;
            for (int ww = 0; ww < kWords; ++ww) n_mem += __popc(members[c][ww]);
            cnt[cl + c] = n_mem;
        }
        cl += P;
        tl = 0;
    } else if (closing) {   // a tail of one token is a cluster of its own, already in place
        cl += tl;
        tl = 0;
    }

    if (is_delim) {   // the delimiter is a chunk of its own: its K/V stay as they are
        __syncthreads();   // its row may be one that another thread was still pooling from
        T* kr = ck + (int64_t)cl * d;
        T* vr = cv + (int64_t)cl * d;
        for (int c = tid; c < d; c += kAppendThreads) { kr[c] = kn[c]; vr[c] = vn[c]; }
        if (tid == 0) cnt[cl] = 1;
        ++cl;
    }
    if (tid == 0) {
        p.core_len[bh] = cl;
        p.tail_len[bh] = tl;
        p.attn_len[bh] = cl + tl;
    }
}

template <typename T>
__global__ void __launch_bounds__(kAppendThreads) append_kernel(const AppendArgs a) {
    LayerPtrs p;
    p.k_new = a.k_new; p.v_new = a.v_new; p.core_k = a.core_k; p.core_v = a.core_v; p.count = a.count;
    p.core_len = a.core_len; p.tail_len = a.tail_len; p.attn_len = a.attn_len;
    append_block<T>(a, p);
}

// Every layer of one generated token in one launch: blockIdx.y picks the layer's row of the table.
template <typename T>
__global__ void __launch_bounds__(kAppendThreads) append_layers_kernel(const AppendArgs a, const sc_append_layer* __restrict__ table) {
    const sc_append_layer t = table[blockIdx.y];
    LayerPtrs p;
    p.k_new = t.k_new; p.v_new = t.v_new; p.core_k = t.core_k; p.core_v = t.core_v; p.count = t.count;
    p.core_len = t.core_len; p.tail_len = t.tail_len; p.attn_len = t.attn_len;
    append_block<T>(a, p);
}

}  // namespace

cudaError_t launch_append_layers(const AppendArgs& a, const sc_append_layer* table, int32_t L, cudaStream_t st) {
    const int blocks = a.B * a.Hkv;
    if (blocks == 0 || L == 0) return cudaSuccess;
    const dim3 grid(blocks, L);
    if (a.dt == SC_BF16) append_layers_kernel<__nv_bfloat16><<<grid, kAppendThreads, 0, st>>>(a, table);
    else append_layers_kernel<float><<<grid, kAppendThreads, 0, st>>>(a, table);
    note_launches(1);
    return cudaGetLastError();
}

cudaError_t launch_append(const AppendArgs& a, cudaStream_t st) {
    const int blocks = a.B * a.Hkv;
    if (blocks == 0) return cudaSuccess;
    if (a.dt == SC_BF16) append_kernel<__nv_bfloat16><<<blocks, kAppendThreads, 0, st>>>(a);
    else append_kernel<float><<<blocks, kAppendThreads, 0, st>>>(a);
    note_launches(1);
    return cudaGetLastError();
}

}  // namespace sc
