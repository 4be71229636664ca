// Tensor-core bf16 decode attention for Eq. 4 (d = 128, query group G <= 8), sm_100a.
//
// One block serves one (sequence, KV head, split): its warps stream 16-row tiles of the head's
// cores through private cp.async rings in shared memory (16-byte chunks, XOR-swizzled so that
// ldmatrix is conflict free) and fold the whole GQA group into one pass:
//     S^T[16 keys x 8 heads]   = K_tile . q^T                (mma.m16n8k16, keys on M, heads on N)
//     x = S^T * scale*log2(e) + log2(count)                  (Proportional Attention, base 2)
//     P^T = 2^(x - m)  (online softmax; the running max is per head and common to the warp)
//     O^T[128 dims x 8 heads] += V_tile^T . P^T              (ldmatrix.trans, P^T via movmatrix)
// Warps are merged in a fixed order through shared memory, the block writes one (m, l, O)
// partial, and the last block of a head to arrive (atomic ticket, no waiting) merges the
// splits in order and writes the output, so results are bit-reproducible.
#include <cstdlib>

#include "common.cuh"

namespace sc {

namespace dm {

// Phase timestamps for a debugging harness; compiled out of the library.
#ifdef SC_TIMELINE
__device__ long long* g_timeline = nullptr;   // [launch][block][16]
__device__ const char* g_timeline_out0 = nullptr;
__device__ long long g_timeline_stride = 1;
#define SC_T(i)                                                                                         \
    do {                                                                                                \
        if (g_timeline && threadIdx.x == 0) {                                                           \
            long long* t_ = g_timeline + ((size_t)tl_launch * 1024 + tl_block) * 16;                    \
            if ((i) == 0) { unsigned long long gt_; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(gt_)); t_[15] = (long long)gt_; } \
            t_[i] = clock64();                                                                          \
        }                                                                                               \
    } while (0)
#else
#define SC_T(i)
#endif

constexpr int kWarps = 4;
constexpr int kStages = 3;
constexpr int kTile = 16;                       // rows per warp tile
constexpr int kD = 128;
constexpr int kRowBytes = kD * 2;               // 256
constexpr int kTileBytes = kTile * kRowBytes;   // 4096 per K or V tile
constexpr int kStageBytes = 2 * kTileBytes + 64;  // K, V, 16 counts
constexpr int kWarpBytes = kStages * kStageBytes;
constexpr int kSmemBytes = kWarps * kWarpBytes;
constexpr int kPartStride = 8 * kD + 16;        // floats per (b, h, split): acc[8 heads][128], m[8], l[8]
constexpr int kCtasPerSm = 2;                   // two kernels (consecutive layers) can be co-resident
constexpr size_t kL2PrefetchBytes = 512 * 1024;  // per tensor and block
constexpr int kCapRowsPerSplit = 1408;           // of capacity (heads are usually half full or less): about 700 rows a block

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, int src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async4(uint32_t dst, const void* src, int src_bytes) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory"); }

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a) {
    uint32_t d;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;\n" : "=r"(d) : "r"(a));
    return d;
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ float bf16_lo(uint32_t v) { return __uint_as_float(v << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t v) { return __uint_as_float(v & 0xffff0000u); }
__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float fast_log2(float x) {
    float y;
    asm("lg2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
    return y;
}

// Copies rows [row0, row0+16) of one head's cores into a stage; rows >= len are zero-filled.
__device__ __forceinline__ void issue_tile(uint32_t stage, const __nv_bfloat16* __restrict__ kh,
                                           const __nv_bfloat16* __restrict__ vh, const int32_t* __restrict__ ch,
                                           int row0, int len, int lane) {
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int idx = i * 32 + lane;          // 256 chunks of 16 B per tile
        const int r = idx >> 4, c = idx & 15;
        const int row = row0 + r;
        const bool ok = row < len;
        const size_t goff = (size_t)(ok ? row : 0) * kD + c * 8;
        const uint32_t soff = r * kRowBytes + ((c ^ (r & 7)) << 4);
        cp_async16(stage + soff, kh + goff, ok ? 16 : 0);
        cp_async16(stage + kTileBytes + soff, vh + goff, ok ? 16 : 0);
    }
    if (ch != nullptr && lane < kTile) {
        const int row = row0 + lane;
        const bool ok = row < len;
        cp_async4(stage + 2 * kTileBytes + lane * 4, ch + (ok ? row : 0), ok ? 4 : 0);
    }
}

__global__ void __launch_bounds__(kWarps * 32, kCtasPerSm)
decode_mma_kernel(const __nv_bfloat16* __restrict__ q, int Hq, int Hkv, const __nv_bfloat16* __restrict__ core_k,
                  const __nv_bfloat16* __restrict__ core_v, const int32_t* __restrict__ count, int cap,
                  const int32_t* __restrict__ core_len, float scale_log2, int n_split,
                  __nv_bfloat16* __restrict__ out, float* __restrict__ part, int32_t* __restrict__ tickets) {
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ float sh_m[kWarps][8];
    __shared__ float sh_l[kWarps][8];
    __shared__ int sh_last;

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g = lane >> 2, tig = lane & 3;
    const int split = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
#ifdef SC_TIMELINE
    const int tl_launch = (int)(((const char*)out - g_timeline_out0) / g_timeline_stride), tl_block = blockIdx.x + gridDim.x * (blockIdx.y + gridDim.y * blockIdx.z);
#endif
    SC_T(0);
    const int G = Hq / Hkv;
    const int bh = b * Hkv + h;
    // Let the next kernel of the stream start beside this one if it was launched with programmatic
    // stream serialization (a no-op otherwise).
    asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory");
    const int len = max(min(core_len[bh], cap), 0);

    SC_T(1);
    const int tiles_total = (len + kTile - 1) / kTile;
    const int tiles_per_split = (tiles_total + n_split - 1) / n_split;
    const int t0 = min(split * tiles_per_split, tiles_total);
    const int t1 = min(t0 + tiles_per_split, tiles_total);
    // this warp's tiles: t0 + warp, t0 + warp + kWarps, ...
    const int my_tiles = (t1 - t0 - warp + kWarps - 1) / kWarps;   // may be <= 0

    const __nv_bfloat16* kh = core_k + (size_t)bh * cap * kD;
    const __nv_bfloat16* vh = core_v + (size_t)bh * cap * kD;
    const int32_t* ch = count ? count + (size_t)bh * cap : nullptr;
    const uint32_t wbase = smem_u32(smem) + warp * kWarpBytes;

    // Ask L2 for this block's whole share up front (bounded), so that under an overlapped launch
    // the HBM reads run while the preceding kernel is still finishing.
    if (threadIdx.x == 0 && t1 > t0) {
        const int r0 = t0 * kTile, r1 = min(t1 * kTile, len);
        size_t bytes = (size_t)(r1 - r0) * kRowBytes;
        if (bytes > kL2PrefetchBytes) bytes = kL2PrefetchBytes;
        const char* pk = reinterpret_cast<const char*>(kh + (size_t)r0 * kD);
        const char* pv = reinterpret_cast<const char*>(vh + (size_t)r0 * kD);
        for (size_t off = 0; off < bytes; off += 65536) {
            const uint32_t sz = (uint32_t)min((size_t)65536, bytes - off);
            asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;\n" ::"l"(pk + off), "r"(sz) : "memory");
            asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;\n" ::"l"(pv + off), "r"(sz) : "memory");
        }
    }

    // prologue: fill the ring
#pragma unroll
    for (int s = 0; s < kStages - 1; ++s) {
        if (s < my_tiles) issue_tile(wbase + s * kStageBytes, kh, vh, ch, (t0 + warp + s * kWarps) * kTile, len, lane);
        cp_async_commit();
    }

    // Under an overlapped launch the caller has promised that the preceding kernel shares no
    // buffer with this call, so nothing is waited for; an ordinary launch is already ordered.
    SC_T(2);
    SC_T(3);

    // q^T as the B operand of every k-step: b0 = q[head g][16ks + 2tig, +1], b1 = same + 8
    uint32_t qb[8][2];
    {
        const __nv_bfloat16* qh = q + ((size_t)b * Hq + (size_t)h * G + g) * kD;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
            qb[ks][0] = (g < G) ? *reinterpret_cast<const uint32_t*>(qh + ks * 16 + 2 * tig) : 0u;
            qb[ks][1] = (g < G) ? *reinterpret_cast<const uint32_t*>(qh + ks * 16 + 2 * tig + 8) : 0u;
        }
    }

    SC_T(4);
    float o[8][4];
#pragma unroll
    for (int mt = 0; mt < 8; ++mt) { o[mt][0] = o[mt][1] = o[mt][2] = o[mt][3] = 0.f; }
    float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;   // heads 2tig and 2tig+1

    // per-lane ldmatrix row/chunk selectors
    const int lm_j = lane >> 3, lm_r = lane & 7;
    const int k_row = lm_r + ((lm_j & 1) << 3), k_csel = lm_j >> 1;    // K: matrices (r0-7,c), (r8-15,c), (r0-7,c+1), (r8-15,c+1)
    const int v_row = lm_r + ((lm_j >> 1) << 3), v_csel = lm_j & 1;    // V^T: (r0-7,c), (r0-7,c+1), (r8-15,c), (r8-15,c+1)

    for (int i = 0; i < my_tiles; ++i) {
        const int pre = i + kStages - 1;
        if (pre < my_tiles)
            issue_tile(wbase + (pre % kStages) * kStageBytes, kh, vh, ch, (t0 + warp + pre * kWarps) * kTile, len, lane);
        cp_async_commit();
        cp_async_wait<kStages - 1>();
        __syncwarp();

        const uint32_t st = wbase + (i % kStages) * kStageBytes;
        const int row0 = (t0 + warp + i * kWarps) * kTile;

        // S^T = K . q^T, two accumulator chains
        float sa[4] = {0.f, 0.f, 0.f, 0.f}, sb[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
            uint32_t a0, a1, a2, a3;
            const int c = 2 * ks + k_csel;
            ldmatrix_x4(st + k_row * kRowBytes + ((c ^ (k_row & 7)) << 4), a0, a1, a2, a3);
            if (ks & 1) mma_bf16(sb, a0, a1, a2, a3, qb[ks][0], qb[ks][1]);
            else mma_bf16(sa, a0, a1, a2, a3, qb[ks][0], qb[ks][1]);
        }
        float lc_lo = 0.f, lc_hi = 0.f;
        if (ch != nullptr) {
            const int* cs = reinterpret_cast<const int*>(smem + warp * kWarpBytes + (i % kStages) * kStageBytes + 2 * kTileBytes);
            lc_lo = fast_log2((float)max(cs[g], 1));
            lc_hi = fast_log2((float)max(cs[g + 8], 1));
        }
        const bool ok_lo = row0 + g < len, ok_hi = row0 + g + 8 < len;
        const float x0 = ok_lo ? fmaf(sa[0] + sb[0], scale_log2, lc_lo) : -INFINITY;
        const float x1 = ok_lo ? fmaf(sa[1] + sb[1], scale_log2, lc_lo) : -INFINITY;
        const float x2 = ok_hi ? fmaf(sa[2] + sb[2], scale_log2, lc_hi) : -INFINITY;
        const float x3 = ok_hi ? fmaf(sa[3] + sb[3], scale_log2, lc_hi) : -INFINITY;
        float mx0 = fmaxf(x0, x2), mx1 = fmaxf(x1, x3);
#pragma unroll
        for (int off = 4; off < 32; off <<= 1) {
            mx0 = fmaxf(mx0, __shfl_xor_sync(kFull, mx0, off));
            mx1 = fmaxf(mx1, __shfl_xor_sync(kFull, mx1, off));
        }
        const float mn0 = fmaxf(m0, mx0), mn1 = fmaxf(m1, mx1);   // finite: a tile has a valid row
        if (__any_sync(kFull, (mn0 != m0) || (mn1 != m1))) {
            const float c0 = fast_exp2(m0 - mn0), c1 = fast_exp2(m1 - mn1);
            l0 *= c0; l1 *= c1;
#pragma unroll
            for (int mt = 0; mt < 8; ++mt) { o[mt][0] *= c0; o[mt][2] *= c0; o[mt][1] *= c1; o[mt][3] *= c1; }
            m0 = mn0; m1 = mn1;
        }
        const uint32_t p_lo = pack_bf16x2(fast_exp2(x0 - m0), fast_exp2(x1 - m1));   // row g
        const uint32_t p_hi = pack_bf16x2(fast_exp2(x2 - m0), fast_exp2(x3 - m1));   // row g + 8
        l0 += bf16_lo(p_lo) + bf16_lo(p_hi);
        l1 += bf16_hi(p_lo) + bf16_hi(p_hi);
        const uint32_t pb0 = movmatrix_trans(p_lo), pb1 = movmatrix_trans(p_hi);

        // O^T += V^T . P^T
#pragma unroll
        for (int mt = 0; mt < 8; ++mt) {
            uint32_t a0, a1, a2, a3;
            const int c = 2 * mt + v_csel;
            ldmatrix_x4_trans(st + kTileBytes + v_row * kRowBytes + ((c ^ (v_row & 7)) << 4), a0, a1, a2, a3);
            mma_bf16(o[mt], a0, a1, a2, a3, pb0, pb1);
        }
        __syncwarp();
    }
    cp_async_wait<0>();
    SC_T(5);

    // ---- merge the warps of this block (fixed order) ----
    // lane-local l covers rows g, g+8 of every tile: sum over the 8 row groups
#pragma unroll
    for (int off = 4; off < 32; off <<= 1) {
        l0 += __shfl_xor_sync(kFull, l0, off);
        l1 += __shfl_xor_sync(kFull, l1, off);
    }
    if (g == 0) {
        sh_m[warp][2 * tig] = m0; sh_m[warp][2 * tig + 1] = m1;
        sh_l[warp][2 * tig] = l0; sh_l[warp][2 * tig + 1] = l1;
    }
    __syncthreads();   // every warp is done with its ring; reuse it as [warp][8 heads][128] fp32
    float bm0 = -INFINITY, bm1 = -INFINITY;
#pragma unroll
    for (int w2 = 0; w2 < kWarps; ++w2) { bm0 = fmaxf(bm0, sh_m[w2][2 * tig]); bm1 = fmaxf(bm1, sh_m[w2][2 * tig + 1]); }
    const float f0 = (m0 == -INFINITY) ? 0.f : fast_exp2(m0 - bm0);
    const float f1 = (m1 == -INFINITY) ? 0.f : fast_exp2(m1 - bm1);
    float* slab = reinterpret_cast<float*>(smem) + warp * (8 * kD);
#pragma unroll
    for (int mt = 0; mt < 8; ++mt) {
        const int d0 = mt * 16 + g;
        slab[(2 * tig) * kD + d0] = o[mt][0] * f0;
        slab[(2 * tig + 1) * kD + d0] = o[mt][1] * f1;
        slab[(2 * tig) * kD + d0 + 8] = o[mt][2] * f0;
        slab[(2 * tig + 1) * kD + d0 + 8] = o[mt][3] * f1;
    }
    __syncthreads();
    float* my_part = part + ((size_t)bh * n_split + split) * kPartStride;
    const float* slabs = reinterpret_cast<const float*>(smem);
    for (int e = threadIdx.x; e < G * kD; e += kWarps * 32) {
        float acc = 0.f;
#pragma unroll
        for (int w2 = 0; w2 < kWarps; ++w2) acc += slabs[w2 * (8 * kD) + e];
        my_part[e] = acc;
    }
    if (threadIdx.x < G) {
        const int hd = threadIdx.x;
        float bm = -INFINITY, bl = 0.f;
#pragma unroll
        for (int w2 = 0; w2 < kWarps; ++w2) bm = fmaxf(bm, sh_m[w2][hd]);
#pragma unroll
        for (int w2 = 0; w2 < kWarps; ++w2) {
            const float mw = sh_m[w2][hd];
            bl += (mw == -INFINITY) ? 0.f : sh_l[w2][hd] * fast_exp2(mw - bm);
        }
        my_part[8 * kD + hd] = bm;
        my_part[8 * kD + 8 + hd] = bl;
    }

    // ---- the last block of this head to arrive merges the splits ----
    SC_T(6);
    __threadfence();
    __syncthreads();
    SC_T(7);
    if (threadIdx.x == 0) {
        const int t = atomicAdd(&tickets[bh], 1);
        sh_last = (t == n_split - 1);
        if (sh_last) tickets[bh] = 0;   // leave the counter ready for the next call
    }
    __syncthreads();
    SC_T(8);
    if (!sh_last) return;
    __threadfence();
    const float* hp = part + (size_t)bh * n_split * kPartStride;
    float* wgt = reinterpret_cast<float*>(smem);            // [n_split][8] weights, then [8] 1/l
    float* lraw = wgt + n_split * 8 + 8;                     // [n_split][8]
    for (int idx = threadIdx.x; idx < n_split * 8; idx += kWarps * 32) {
        const int s = idx >> 3, hd = idx & 7;
        wgt[idx] = __ldcg(hp + (size_t)s * kPartStride + 8 * kD + hd);
        lraw[idx] = __ldcg(hp + (size_t)s * kPartStride + 8 * kD + 8 + hd);
    }
    __syncthreads();
    if (threadIdx.x < 8) {
        const int hd = threadIdx.x;
        float gm = -INFINITY;
        for (int s = 0; s < n_split; ++s) gm = fmaxf(gm, wgt[s * 8 + hd]);
        float lsum = 0.f;
        for (int s = 0; s < n_split; ++s) {
            const float ms = wgt[s * 8 + hd];
            const float w = (ms == -INFINITY) ? 0.f : fast_exp2(ms - gm);
            wgt[s * 8 + hd] = w;
            lsum = fmaf(w, lraw[s * 8 + hd], lsum);
        }
        wgt[n_split * 8 + hd] = lsum > 0.f ? 1.f / lsum : 0.f;
    }
    __syncthreads();
    for (int e4 = threadIdx.x; e4 < G * (kD / 4); e4 += kWarps * 32) {
        const int hd = e4 / (kD / 4), d4 = (e4 % (kD / 4)) * 4;
        const float* src = hp + hd * kD + d4;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 8
        for (int s = 0; s < n_split; ++s) {
            const float4 v = __ldcg(reinterpret_cast<const float4*>(src + (size_t)s * kPartStride));
            const float w = wgt[s * 8 + hd];
            acc.x = fmaf(w, v.x, acc.x); acc.y = fmaf(w, v.y, acc.y);
            acc.z = fmaf(w, v.z, acc.z); acc.w = fmaf(w, v.w, acc.w);
        }
        const float inv = wgt[n_split * 8 + hd];
        __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x * inv, acc.y * inv);
        __nv_bfloat162 hi = __floats2bfloat162_rn(acc.z * inv, acc.w * inv);
        uint2 pk;
        pk.x = *reinterpret_cast<uint32_t*>(&lo);
        pk.y = *reinterpret_cast<uint32_t*>(&hi);
        *reinterpret_cast<uint2*>(out + ((size_t)b * Hq + (size_t)h * G + hd) * kD + d4) = pk;
    }
    SC_T(9);
}

inline int splits_for(int B, int Hkv, int cap, int sms) {
    const int heads = B * Hkv;
    int s = sms / heads;   // one block per SM, so the next layer's blocks fit beside this one's
    // ... unless that leaves a block thousands of rows to stream alone (many heads, long caches): then several
    // waves of shorter blocks keep HBM busier (measured: 0.81 -> 1.06 of the copy peak at 128 heads x 8K rows)
    const int by_len = (cap + kCapRowsPerSplit - 1) / kCapRowsPerSplit;
    if (by_len > s) s = by_len;
    const int max_by_rows = (cap + 4 * kTile - 1) / (4 * kTile);   // at least 64 rows per split
    if (s > max_by_rows) s = max_by_rows;
    if (s > 256) s = 256;
    return s < 1 ? 1 : s;
}

}  // namespace dm

bool decode_mma_supported(const DecodeArgs& a) {
    return a.dt == SC_BF16 && a.d == dm::kD && (a.Hq / a.Hkv) <= 8 && a.cap > 0 && a.Hkv <= 65535 && a.B <= 65535;
}

size_t decode_mma_ws_bytes(int32_t B, int32_t Hq, int32_t Hkv, int32_t d, int32_t cap) {
    (void)Hq; (void)d;
    // tickets (one per (b, head), zero between calls) + partials for the largest split count
    const int s = dm::splits_for(B, Hkv, cap, 256);
    const int s2 = dm::splits_for(B, Hkv, cap, 132);
    int smax = s > s2 ? s : s2;
#ifdef SC_TUNE
    if (smax < 64) smax = 64;
#endif
    return 256 + sizeof(int32_t) * (((size_t)B * Hkv + 63) / 64 * 64) +
           sizeof(float) * (size_t)B * Hkv * smax * dm::kPartStride;
}

cudaError_t launch_decode_mma(const DecodeArgs& a, cudaStream_t st) {
    static int sms_of[64] = {0};   // per device: SM count, and the opt-in to large dynamic shared memory
    int dev = 0;
    cudaGetDevice(&dev);
    dev &= 63;
    if (sms_of[dev] == 0) {
        int v = 0;
        cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev);
        cudaFuncSetAttribute(dm::decode_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, dm::kSmemBytes);
        sms_of[dev] = v > 256 ? 256 : (v < 1 ? 1 : v);
    }
    const int sms = sms_of[dev];
    int n_split = dm::splits_for(a.B, a.Hkv, a.cap, sms);
#ifdef SC_TUNE   // tuning harness only
    if (const char* e = getenv("SC_DEC_SPLITS")) n_split = atoi(e);
#endif
    int32_t* tickets = (int32_t*)a.ws;
    float* part = (float*)((char*)a.ws + sizeof(int32_t) * (((size_t)a.B * a.Hkv + 63) / 64 * 64));
    const float scale = (a.scale == 0.f ? 1.f / sqrtf((float)a.d) : a.scale) * 1.4426950408889634f;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(n_split, a.Hkv, a.B);
    cfg.blockDim = dim3(dm::kWarps * 32);
    cfg.dynamicSmemBytes = dm::kSmemBytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = (a.flags & SC_FLAG_OVERLAP_PREV) ? 1 : 0;
    note_launches(1);
    return cudaLaunchKernelEx(&cfg, dm::decode_mma_kernel, (const __nv_bfloat16*)a.q, a.Hq, a.Hkv,
                              (const __nv_bfloat16*)a.core_k, (const __nv_bfloat16*)a.core_v, a.count, a.cap,
                              a.core_len, scale, n_split, (__nv_bfloat16*)a.out, part, tickets);
}

}  // namespace sc
