// Generic decode path for Eq. 4 (any dtype, d <= 256 multiple of 8): one warp per
// (sequence, query head, split) streams its share of the cores with an online softmax in fp32,
// then a second kernel combines the splits in order.  Serves SC_F32 and cross-checks the
// tensor-core bf16 kernel.
#include "common.cuh"

namespace sc {

constexpr int kDecWarps = 4;
constexpr int kMaxPerLaneD = 8;

__host__ __device__ inline int generic_splits(int cap) {
    int s = (cap + 511) / 512;
    return s < 1 ? 1 : (s > 64 ? 64 : s);
}

template <typename T>
__global__ void __launch_bounds__(kDecWarps * 32)
decode_generic(const T* __restrict__ q, int B, int Hq, int Hkv, int d, const T* __restrict__ core_k,
               const T* __restrict__ core_v, const int32_t* __restrict__ count, int cap,
               const int32_t* __restrict__ core_len, float scale_log2, int n_split, float* __restrict__ part) {
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int64_t items = (int64_t)B * Hq * n_split;
    const int64_t it = (int64_t)blockIdx.x * kDecWarps + w;
    if (it >= items) return;
    const int sp = (int)(it % n_split);
    const int hq = (int)((it / n_split) % Hq);
    const int b = (int)(it / ((int64_t)n_split * Hq));
    const int G = Hq / Hkv, h = hq / G;
    const int len = min(core_len[b * Hkv + h], cap);
    const int per_split = (len + n_split - 1) / n_split;
    const int t0 = min(sp * per_split, len), t1 = min(t0 + per_split, len);
    const T* qr = q + ((int64_t)b * Hq + hq) * d;
    const int64_t cbase = ((int64_t)b * Hkv + h) * cap;
    float qv[kMaxPerLaneD], acc[kMaxPerLaneD];
#pragma unroll
    for (int u = 0; u < kMaxPerLaneD; ++u) {
        int c = lane + 32 * u;
        qv[u] = (c < d) ? Elem<T>::load(qr + c) * scale_log2 : 0.f;
        acc[u] = 0.f;
    }
    float m = -INFINITY, lsum = 0.f;
    for (int t = t0; t < t1; ++t) {
        const T* kr = core_k + (cbase + t) * d;
        const T* vr = core_v + (cbase + t) * d;
        float s = 0.f;
#pragma unroll
        for (int u = 0; u < kMaxPerLaneD; ++u) {
            int c = lane + 32 * u;
            if (c < d) s = fmaf(qv[u], Elem<T>::load(kr + c), s);
        }
        s = warp_sum(s);
        if (count != nullptr) s += log2f((float)max(count[cbase + t], 1));  // ln s, in base-2 units (a valid row has count >= 1)
        const float mn = fmaxf(m, s);
        const float corr = exp2f(m - mn);  // m = -inf on the first row gives 0
        const float pw = exp2f(s - mn);
        lsum = lsum * corr + pw;
#pragma unroll
        for (int u = 0; u < kMaxPerLaneD; ++u) {
            int c = lane + 32 * u;
            if (c < d) acc[u] = acc[u] * corr + pw * Elem<T>::load(vr + c);
        }
        m = mn;
    }
    float* pr = part + it * (d + 2);
#pragma unroll
    for (int u = 0; u < kMaxPerLaneD; ++u) {
        int c = lane + 32 * u;
        if (c < d) pr[c] = acc[u];
    }
    if (lane == 0) { pr[d] = m; pr[d + 1] = lsum; }
}

template <typename T>
__global__ void __launch_bounds__(kDecWarps * 32)
combine_generic(int64_t heads, int d, int n_split, const float* __restrict__ part, T* __restrict__ out) {
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int64_t hd = (int64_t)blockIdx.x * kDecWarps + w;
    if (hd >= heads) return;
    const float* pr = part + hd * n_split * (d + 2);
    float m = -INFINITY;
    for (int s = 0; s < n_split; ++s) m = fmaxf(m, pr[s * (d + 2) + d]);
    float acc[kMaxPerLaneD];
#pragma unroll
    for (int u = 0; u < kMaxPerLaneD; ++u) acc[u] = 0.f;
    float lsum = 0.f;
    for (int s = 0; s < n_split; ++s) {
        const float ms = pr[s * (d + 2) + d];
        if (ms == -INFINITY) continue;  // an empty split
        const float wgt = exp2f(ms - m);
        lsum += wgt * pr[s * (d + 2) + d + 1];
#pragma unroll
        for (int u = 0; u < kMaxPerLaneD; ++u) {
            int c = lane + 32 * u;
            if (c < d) acc[u] += wgt * pr[s * (d + 2) + c];
        }
    }
    const float inv = lsum > 0.f ? 1.f / lsum : 0.f;
#pragma unroll
    for (int u = 0; u < kMaxPerLaneD; ++u) {
        int c = lane + 32 * u;
        if (c < d) Elem<T>::store(out + hd * d + c, acc[u] * inv);
    }
}

size_t decode_generic_ws_bytes(int32_t B, int32_t Hq, int32_t Hkv, int32_t d, int32_t cap) {
    (void)Hkv;
    return sizeof(float) * (size_t)B * Hq * generic_splits(cap) * (d + 2) + 256;
}

template <typename T>
static cudaError_t run(const DecodeArgs& a, cudaStream_t st) {
    const int n_split = generic_splits(a.cap);
    const int64_t items = (int64_t)a.B * a.Hq * n_split;
    const float scale = (a.scale == 0.f ? 1.f / sqrtf((float)a.d) : a.scale) * 1.4426950408889634f;
    decode_generic<T><<<div_up(items, kDecWarps), kDecWarps * 32, 0, st>>>(
        (const T*)a.q, a.B, a.Hq, a.Hkv, a.d, (const T*)a.core_k, (const T*)a.core_v, a.count, a.cap, a.core_len,
        scale, n_split, (float*)a.ws);
    const int64_t heads = (int64_t)a.B * a.Hq;
    combine_generic<T><<<div_up(heads, kDecWarps), kDecWarps * 32, 0, st>>>(heads, a.d, n_split, (const float*)a.ws,
                                                                          (T*)a.out);
    note_launches(2);
    return cudaGetLastError();
}

cudaError_t launch_decode_generic(const DecodeArgs& a, cudaStream_t st) {
    return a.dt == SC_BF16 ? run<__nv_bfloat16>(a, st) : run<float>(a, st);
}

}  // namespace sc
