// Generic compress path (any dtype, any d <= 256 that is a multiple of 8, any strides):
// three kernels per layer -- GSC per segment, prefix sum of cluster counts per (b, head),
// mean-pool merge per segment.  CUDA-core arithmetic in fp32; serves SC_F32 and is the
// cross-check of the fused bf16 path.
#include "common.cuh"

namespace sc {

constexpr int kGenWarps = 8;
constexpr int kMaxPerLane = 8;  // d <= 256

// Algorithm 1 for one segment per warp.  Keys are read straight from global memory; the seed
// row is held in registers and each candidate row is dotted against it across the warp.
template <typename T>
__global__ void __launch_bounds__(kGenWarps * 32)
gsc_generic(const T* __restrict__ K, sc_strides st, int B, int Hkv, int n, int d,
            const int32_t* __restrict__ seg_off, const int32_t* __restrict__ n_seg_p, int seg_stride,
            float tau_host, const float* __restrict__ tau_dev, const int32_t* __restrict__ skip,
            int32_t* __restrict__ assign, int32_t* __restrict__ seg_p) {
    __shared__ float norms[kGenWarps][SC_MAX_CHUNK_LEN];
    if (skip != nullptr && *skip != 0) return;
    const float tau = tau_dev != nullptr ? *tau_dev : tau_host;
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int n_seg = min(*n_seg_p, seg_stride);
    const int64_t items = (int64_t)n_seg * Hkv;
    const int per = d / 32 + ((d % 32) ? 1 : 0);
    for (int64_t it = (int64_t)blockIdx.x * kGenWarps + w; it < items; it += (int64_t)gridDim.x * kGenWarps) {
        const int s = (int)(it % n_seg), h = (int)(it / n_seg);
        const int a = seg_off[s], e = seg_off[s + 1];
        const int b = a / n, r = a - b * n, l = min(e - a, SC_MAX_CHUNK_LEN);
        const T* Kb = K + b * st.b + h * st.h;
        int32_t* as = assign + ((int64_t)b * Hkv + h) * n;
        // norms
        for (int i = 0; i < l; ++i) {
            const T* row = Kb + (int64_t)(r + i) * st.n;
            float acc = 0.f;
            for (int c = lane; c < d; c += 32) { float x = Elem<T>::load(row + c); acc = fmaf(x, x, acc); }
            acc = warp_sum(acc);
            if (lane == 0) norms[w][i] = sqrtf(acc);
        }
        __syncwarp();
        unsigned word = 0;  // lane c holds the assigned bits of tokens 32c .. 32c+31
        int p = 0;
        for (int i = 0; i < l; ++i) {
            unsigned wi = __shfl_sync(kFull, word, i >> 5);
            if ((wi >> (i & 31)) & 1u) continue;
            ++p;
            if (lane == (i >> 5)) word |= 1u << (i & 31);
            if (lane == 0) as[r + i] = r + i;
            float seed[kMaxPerLane];
            const T* srow = Kb + (int64_t)(r + i) * st.n;
#pragma unroll
            for (int u = 0; u < kMaxPerLane; ++u) {
                int c = lane + 32 * u;
                seed[u] = (u < per && c < d) ? Elem<T>::load(srow + c) : 0.f;
            }
            const float ni = norms[w][i];
            for (int j = i + 1; j < l; ++j) {
                unsigned wj = __shfl_sync(kFull, word, j >> 5);
                if ((wj >> (j & 31)) & 1u) continue;
                const T* row = Kb + (int64_t)(r + j) * st.n;
                float acc = 0.f;
#pragma unroll
                for (int u = 0; u < kMaxPerLane; ++u) {
                    int c = lane + 32 * u;
                    if (u < per && c < d) acc = fmaf(seed[u], Elem<T>::load(row + c), acc);
                }
                acc = warp_sum(acc);
                const float nj = norms[w][j];
                const float sim = (ni == 0.f || nj == 0.f) ? 0.f : acc / (ni * nj);
                if (sim > tau) {
                    if (lane == (j >> 5)) word |= 1u << (j & 31);
                    if (lane == 0) as[r + j] = r + i;
                }
            }
        }
        if (lane == 0) seg_p[(int64_t)h * seg_stride + s] = p;
        __syncwarp();
    }
}

// Exclusive prefix sum of the per-segment cluster counts inside each (b, head).
__global__ void __launch_bounds__(256)
scan_generic(int Hkv, const int32_t* __restrict__ seq_seg_off, int seg_stride,
             const int32_t* __restrict__ seg_p, int32_t* __restrict__ seg_core_off,
             int32_t* __restrict__ core_len, int cap, int32_t* status, const int32_t* __restrict__ skip,
             int count_only) {
    __shared__ int wt[8];
    if (skip != nullptr && *skip != 0) return;
    const int b = blockIdx.x / Hkv, h = blockIdx.x % Hkv;
    const int s0 = min(seq_seg_off[b], seg_stride), s1 = min(seq_seg_off[b + 1], seg_stride);
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    int carry = 0;
    for (int base = s0; base < s1; base += 256) {
        int s = base + threadIdx.x;
        int v = (s < s1) ? seg_p[(int64_t)h * seg_stride + s] : 0;
        int incl = warp_scan_add(v, lane);
        if (lane == 31) wt[w] = incl;
        __syncthreads();
        int pre = 0, tot = 0;
        for (int i = 0; i < 8; ++i) { if (i < w) pre += wt[i]; tot += wt[i]; }
        __syncthreads();
        if (s < s1) seg_core_off[(int64_t)h * seg_stride + s] = carry + pre + incl - v;
        carry += tot;
    }
    if (threadIdx.x == 0) {
        core_len[b * Hkv + h] = carry;
        if (carry > cap && !count_only) set_status(status, SC_ERR_CAPACITY);
    }
}

// Eq. 3 for one segment per warp: fp32 sums in token order, one divide, one rounding.
template <typename T>
__global__ void __launch_bounds__(kGenWarps * 32)
merge_generic(const T* __restrict__ K, const T* __restrict__ V, sc_strides st, int B, int Hkv, int n, int d,
              const int32_t* __restrict__ seg_off, const int32_t* __restrict__ n_seg_p, int seg_stride,
              const int32_t* __restrict__ assign, const int32_t* __restrict__ seg_core_off,
              T* __restrict__ core_k, T* __restrict__ core_v, int32_t* __restrict__ count, int cap) {
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int n_seg = min(*n_seg_p, seg_stride);
    const int64_t items = (int64_t)n_seg * Hkv;
    for (int64_t it = (int64_t)blockIdx.x * kGenWarps + w; it < items; it += (int64_t)gridDim.x * kGenWarps) {
        const int s = (int)(it % n_seg), h = (int)(it / n_seg);
        const int a = seg_off[s], e = seg_off[s + 1];
        const int b = a / n, r = a - b * n, l = min(e - a, SC_MAX_CHUNK_LEN);
        const T* Kb = K + b * st.b + h * st.h;
        const T* Vb = V + b * st.b + h * st.h;
        const int32_t* as = assign + ((int64_t)b * Hkv + h) * n;
        int row = seg_core_off[(int64_t)h * seg_stride + s];
        const int64_t obase = ((int64_t)b * Hkv + h) * cap;
        for (int i = 0; i < l; ++i) {
            if (as[r + i] != r + i) continue;
            float sk[kMaxPerLane], sv[kMaxPerLane];
#pragma unroll
            for (int u = 0; u < kMaxPerLane; ++u) sk[u] = sv[u] = 0.f;
            int cnt = 0;
            for (int j = i; j < l; ++j) {
                if (as[r + j] != r + i) continue;
                ++cnt;
                const T* kr = Kb + (int64_t)(r + j) * st.n;
                const T* vr = Vb + (int64_t)(r + j) * st.n;
#pragma unroll
                for (int u = 0; u < kMaxPerLane; ++u) {
                    int c = lane + 32 * u;
                    if (c < d) { sk[u] += Elem<T>::load(kr + c); sv[u] += Elem<T>::load(vr + c); }
                }
            }
            if (row < cap) {
                const float fc = (float)cnt;
#pragma unroll
                for (int u = 0; u < kMaxPerLane; ++u) {
                    int c = lane + 32 * u;
                    if (c < d) {
                        Elem<T>::store(core_k + (obase + row) * d + c, sk[u] / fc);
                        Elem<T>::store(core_v + (obase + row) * d + c, sv[u] / fc);
                    }
                }
                if (lane == 0) count[obase + row] = cnt;
            }
            ++row;
        }
    }
}

size_t compress_generic_ws_bytes(int32_t B, int32_t Hkv, int32_t n) {
    // assign (when the caller passes none) + seg_p + seg_core_off, each B*Hkv*n int32
    return sizeof(int32_t) * 3 * (size_t)B * Hkv * n + 256;
}

template <typename T>
static cudaError_t run(const CompressArgs& a, cudaStream_t st) {
    const size_t per = (size_t)a.B * a.Hkv * a.n;
    int32_t* ws = (int32_t*)a.ws;
    int32_t* seg_p = ws;
    int32_t* seg_core_off = ws + per;
    int32_t* assign = (a.assign && !a.count_only) ? a.assign : ws + 2 * per;
    const int seg_stride = a.B * a.n;  // capacity of the segment axis
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const int grid = sms * 8;
    gsc_generic<T><<<grid, kGenWarps * 32, 0, st>>>((const T*)a.K, a.st, a.B, a.Hkv, a.n, a.d, a.seg_off, a.n_seg,
                                                    seg_stride, a.tau, a.tau_dev, a.skip, assign, seg_p);
    scan_generic<<<a.B * a.Hkv, 256, 0, st>>>(a.Hkv, a.seq_seg_off, seg_stride, seg_p, seg_core_off, a.core_len,
                                              a.cap, a.status, a.skip, a.count_only);
    if (a.count_only) {   // budget search: per-head cluster counts only
        note_launches(2);
        return cudaGetLastError();
    }
    merge_generic<T><<<grid, kGenWarps * 32, 0, st>>>((const T*)a.K, (const T*)a.V, a.st, a.B, a.Hkv, a.n, a.d,
                                                      a.seg_off, a.n_seg, seg_stride, assign, seg_core_off,
                                                      (T*)a.core_k, (T*)a.core_v, a.count, a.cap);
    note_launches(3);
    return cudaGetLastError();
}

cudaError_t launch_compress_generic(const CompressArgs& a, cudaStream_t st) {
    return a.dt == SC_BF16 ? run<__nv_bfloat16>(a, st) : run<float>(a, st);
}

}  // namespace sc
