// Tensor-core bf16 decode attention for Eq. 4 (d = 128, query group G <= 8), sm_100a.
//
// One block serves one (sequence, KV head, split): its warps stream 16-row tiles of the head's
// cores through private cp.async rings in shared memory (16-byte chunks, XOR-swizzled so that
// ldmatrix is conflict free) and fold the whole GQA group into one pass:
//     S^T[16 keys x 8 heads]   = K_tile . q^T                (mma.m16n8k16, keys on M, heads on N)
//     x = S^T * scale*log2(e) + log2(count)                  (Proportional Attention, base 2)
//     P^T = 2^(x - m)  (online softmax; the running max is per head, common to the warp, and
//                       raised only when a score overtakes it by a margin)
//     O^T[128 dims x 8 heads] += V_tile^T . P^T              (ldmatrix.trans, P^T via movmatrix,
//                                                             as a bf16 pair: leading part + remainder)
// Warps are merged in a fixed order through shared memory into one (m, l, O) partial per block.
// When the launch is about one wave of blocks, the splits of a head form a thread-block cluster
// and fold their partials through distributed shared memory, each block its own slice of the
// output (no partial leaves the SMs); otherwise, or when a head needs several clusters, partials go
// to global memory and the last block of a head to arrive (atomic ticket, no waiting) merges them.
// In such a launch of several waves the split count comes from the capacity, which the host knows; how many of
// those blocks a head really uses is settled by each block from the head's length (about 1024 rows a block, 768 in the largest launches, but
// enough blocks over the launch to fill the GPU three times): the others take their ticket and leave.
// Every order is fixed, so results are bit-reproducible.
//
// Launch modes: ordinary; overlapped with the preceding kernel (programmatic stream
// serialization), where every global write waits for that kernel's completion; and chained, where
// in addition q is read only after that wait (q is the preceding kernel's product) while the cores
// were requested before it.
#include <cooperative_groups.h>

#include "common.cuh"

namespace sc {

namespace dm {

namespace cg = cooperative_groups;

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
constexpr float kMaxSlack = 8.f;                // log2 units a score may exceed the running maximum before it is raised
constexpr int kMergeGroup = 16;                 // cluster partials folded per round by the merging block
constexpr int kMaxCluster = 16;                 // blocks per cluster (more than 8 needs the non-portable opt-in)
constexpr int kRowsPerBlock = 1024;              // rows a block should stream at least, where the head's length allows ...
constexpr int kRowsPerBlockBig = 768;            // ... in a launch over kBigLaunchRows rows of capacity (more, shorter blocks keep HBM busier there)
constexpr long long kBigLaunchRows = 1300000;
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

__device__ __forceinline__ void store_out4(__nv_bfloat16* dst, const float4& acc, float inv) {
    __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x * inv, acc.y * inv);
    __nv_bfloat162 hi = __floats2bfloat162_rn(acc.z * inv, acc.w * inv);
    uint2 pk;
    pk.x = *reinterpret_cast<uint32_t*>(&lo);
    pk.y = *reinterpret_cast<uint32_t*>(&hi);
    *reinterpret_cast<uint2*>(dst) = pk;
}

// Copies rows [row0, row0+16) of one head's cores into a stage; rows >= len are zero-filled.  Lane l
// moves 16-byte chunk l & 15 of rows 2i + (l >> 4), i = 0..7, to its swizzled place soff[i] (the same
// for every tile, so the caller computes the eight offsets once).  A tile that lies wholly inside the
// head -- all but the last one -- needs no per-row test.
__device__ __forceinline__ void issue_tile(uint32_t stage, const __nv_bfloat16* __restrict__ kh,
                                           const __nv_bfloat16* __restrict__ vh, const int32_t* __restrict__ ch,
                                           int row0, int len, int lane, const uint32_t (&soff)[8]) {
    const size_t g0 = (size_t)(row0 + (lane >> 4)) * kD + (lane & 15) * 8;
    if (row0 + kTile <= len) {
        const __nv_bfloat16* ks = kh + g0;
        const __nv_bfloat16* vs = vh + g0;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            cp_async16(stage + soff[i], ks + i * 2 * kD, 16);
            cp_async16(stage + kTileBytes + soff[i], vs + i * 2 * kD, 16);
        }
        if (ch != nullptr && lane < kTile) cp_async4(stage + 2 * kTileBytes + lane * 4, ch + row0 + lane, 4);
        return;
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const bool ok = row0 + 2 * i + (lane >> 4) < len;
        const size_t goff = ok ? g0 + (size_t)i * 2 * kD : 0;
        cp_async16(stage + soff[i], kh + goff, ok ? 16 : 0);
        cp_async16(stage + kTileBytes + soff[i], vh + goff, ok ? 16 : 0);
    }
    if (ch != nullptr && lane < kTile) {
        const int row = row0 + lane;
        const bool ok = row < len;
        cp_async4(stage + 2 * kTileBytes + lane * 4, ch + (ok ? row : 0), ok ? 4 : 0);
    }
}

// Several partials per head in global memory (one per cluster, or per block outside clusters): the last block
// to arrive merges the first `n_parts` of them (the others belong to blocks that found no tiles).  All threads of
// the block call it.  The cluster barrier / fence before the call orders this block's partial stores before its
// ticket, whose release makes them visible to whoever reads the ticket with acquire (the last arrival); that
// block's other threads are ordered behind its thread 0 by the barrier below and read the partials from L2.
__device__ __forceinline__ void ticket_and_merge(const float* __restrict__ part, int32_t* __restrict__ tickets, int bh,
                                                 int n_expected, int n_parts, int G, int Hq, int b, int h,
                                                 __nv_bfloat16* __restrict__ out, int* sh_last_p) {
    if (threadIdx.x == 0) {
        int t;
        asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], 1;\n" : "=r"(t) : "l"(tickets + bh) : "memory");
        *sh_last_p = (t == n_expected - 1);
        if (*sh_last_p) tickets[bh] = 0;   // leave the counter ready for the next call
    }
    __syncthreads();
    if (!*sh_last_p) return;
    // One thread per (head, four output columns); the partials are folded sixteen at a time, all of a
    // group's loads in flight together (one round trip to L2 per group).
    const float* hp = part + (size_t)bh * n_expected * kPartStride;
    for (int e4 = threadIdx.x; e4 < G * (kD / 4); e4 += kWarps * 32) {
        const int hd = e4 / (kD / 4), d4 = (e4 % (kD / 4)) * 4;
        float gm = -INFINITY, lsum = 0.f;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int s0 = 0; s0 < n_parts; s0 += kMergeGroup) {
            float mv[kMergeGroup], lv[kMergeGroup];
            float4 ov[kMergeGroup];
#pragma unroll
            for (int j = 0; j < kMergeGroup; ++j) {
                const bool ok = s0 + j < n_parts;
                const float* sp = hp + (size_t)(ok ? s0 + j : 0) * kPartStride;
                mv[j] = ok ? __ldcg(sp + 8 * kD + hd) : -INFINITY;
                lv[j] = ok ? __ldcg(sp + 8 * kD + 8 + hd) : 0.f;
                ov[j] = ok ? __ldcg(reinterpret_cast<const float4*>(sp + hd * kD + d4)) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
            float cm = mv[0];
#pragma unroll
            for (int j = 1; j < kMergeGroup; ++j) cm = fmaxf(cm, mv[j]);
            const float ngm = fmaxf(gm, cm);
            if (ngm == -INFINITY) continue;   // nothing but empty splits so far
            const float c = (gm == -INFINITY) ? 0.f : fast_exp2(gm - ngm);
            lsum *= c; acc.x *= c; acc.y *= c; acc.z *= c; acc.w *= c;
            gm = ngm;
#pragma unroll
            for (int j = 0; j < kMergeGroup; ++j) {
                const float w = (mv[j] == -INFINITY) ? 0.f : fast_exp2(mv[j] - gm);
                lsum = fmaf(w, lv[j], lsum);
                acc.x = fmaf(w, ov[j].x, acc.x); acc.y = fmaf(w, ov[j].y, acc.y);
                acc.z = fmaf(w, ov[j].z, acc.z); acc.w = fmaf(w, ov[j].w, acc.w);
            }
        }
        const float inv = lsum > 0.f ? 1.f / lsum : 0.f;
        store_out4(out + ((size_t)b * Hq + (size_t)h * G + hd) * kD + d4, acc, inv);
    }
}

__global__ void __launch_bounds__(kWarps * 32, kCtasPerSm)
decode_mma_kernel(const __nv_bfloat16* __restrict__ q, int Hq, int Hkv, const __nv_bfloat16* __restrict__ core_k,
                  const __nv_bfloat16* __restrict__ core_v, const int32_t* __restrict__ count, int cap,
                  const int32_t* __restrict__ core_len, float scale_log2, int n_split, int min_split, int rows_block, int q_from_prev,
                  __nv_bfloat16* __restrict__ out, float* __restrict__ part, int32_t* __restrict__ tickets) {
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ float sh_m[kWarps][8];
    __shared__ float sh_l[kWarps][8];
    __shared__ int sh_last;

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g = lane >> 2, tig = lane & 3;
    const int split = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
    const int G = Hq / Hkv;
    const int bh = b * Hkv + h;
    // Let the next kernel of the stream start beside this one if it was launched with programmatic
    // stream serialization (a no-op otherwise).  Whatever this block reads before its own
    // griddepcontrol.wait below (core_len, cores, counts) must not be written by a kernel that may
    // still be running then; that is the caller's promise when it asks for an overlapped launch.
    asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory");
    const int len = max(min(core_len[bh], cap), 0);
    const int tiles_total = (len + kTile - 1) / kTile;
    // The split count was chosen from the capacity; a head that is far from full is shared out among fewer blocks
    // (about rows_block rows each: shorter blocks are mostly prologue and merge), the others find no tiles and
    // hand in an empty partial.  Not inside a cluster, whose blocks are few and fold on chip.
    int eff_split = n_split;
    if (cg::this_cluster().num_blocks() == 1) eff_split = min(n_split, max(min_split, (len + rows_block - 1) / rows_block));
    const int tiles_per_split = (tiles_total + eff_split - 1) / eff_split;
    if (split >= eff_split) {   // a block without tiles: it only takes its ticket (and merges, if it is the last)
        asm volatile("griddepcontrol.wait;\n" ::: "memory");   // no global write before the preceding kernel is complete
        ticket_and_merge(part, tickets, bh, n_split, eff_split, G, Hq, b, h, out, &sh_last);
        return;
    }
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

    uint32_t soff[8];   // this lane's eight chunk places inside a K or V tile (see issue_tile)
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int r = 2 * i + (lane >> 4), c = lane & 15;
        soff[i] = r * kRowBytes + ((c ^ (r & 7)) << 4);
    }

    // prologue: fill the whole ring (under a chained launch this is what is in shared memory when the wait ends)
#pragma unroll
    for (int s = 0; s < kStages; ++s) {
        if (s < my_tiles) issue_tile(wbase + s * kStageBytes, kh, vh, ch, (t0 + warp + s * kWarps) * kTile, len, lane, soff);
        cp_async_commit();
    }

    // Chained launch (SC_FLAG_OVERLAP_CHAIN): q is the preceding kernel's product.  The cores' first
    // tiles are on their way to shared memory and the rest of the block's share to L2; only now wait
    // for that kernel to complete (and its writes to be visible), then read q.
    if (q_from_prev) asm volatile("griddepcontrol.wait;\n" ::: "memory");

    // q^T as the B operand of every k-step: b0 = q[head g][16ks + 2tig, +1], b1 = same + 8
    uint32_t qb[8][2];
    {
        const __nv_bfloat16* qh = q + ((size_t)b * Hq + (size_t)h * G + g) * kD;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
            // read through L2: under a chained launch q was written while this kernel was already running
            qb[ks][0] = (g < G) ? __ldcg(reinterpret_cast<const uint32_t*>(qh + ks * 16 + 2 * tig)) : 0u;
            qb[ks][1] = (g < G) ? __ldcg(reinterpret_cast<const uint32_t*>(qh + ks * 16 + 2 * tig + 8)) : 0u;
        }
    }
    float o[8][4];
#pragma unroll
    for (int mt = 0; mt < 8; ++mt) { o[mt][0] = o[mt][1] = o[mt][2] = o[mt][3] = 0.f; }
    float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;   // heads 2tig and 2tig+1

    // per-lane ldmatrix row/chunk selectors
    const int lm_j = lane >> 3, lm_r = lane & 7;
    const int k_row = lm_r + ((lm_j & 1) << 3), k_csel = lm_j >> 1;    // K: matrices (r0-7,c), (r8-15,c), (r0-7,c+1), (r8-15,c+1)
    const int v_row = lm_r + ((lm_j >> 1) << 3), v_csel = lm_j & 1;    // V^T: (r0-7,c), (r0-7,c+1), (r8-15,c), (r8-15,c+1)

    for (int i = 0; i < my_tiles; ++i) {
        cp_async_wait<kStages - 1>();   // tile i has landed; tiles i+1, i+2 are on their way
        __syncwarp();

        const uint32_t st = wbase + (i % kStages) * kStageBytes;
        const int row0 = (t0 + warp + i * kWarps) * kTile;

        // S^T = K . q^T, four accumulator chains
        float sa[4] = {0.f, 0.f, 0.f, 0.f}, sb[4] = {0.f, 0.f, 0.f, 0.f};
        float sc2[4] = {0.f, 0.f, 0.f, 0.f}, sd[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
            uint32_t a0, a1, a2, a3;
            const int c = 2 * ks + k_csel;
            ldmatrix_x4(st + k_row * kRowBytes + ((c ^ (k_row & 7)) << 4), a0, a1, a2, a3);
            if ((ks & 3) == 0) mma_bf16(sa, a0, a1, a2, a3, qb[ks][0], qb[ks][1]);
            else if ((ks & 3) == 1) mma_bf16(sb, a0, a1, a2, a3, qb[ks][0], qb[ks][1]);
            else if ((ks & 3) == 2) mma_bf16(sc2, a0, a1, a2, a3, qb[ks][0], qb[ks][1]);
            else mma_bf16(sd, a0, a1, a2, a3, qb[ks][0], qb[ks][1]);
        }
        float lc_lo = 0.f, lc_hi = 0.f;
        if (ch != nullptr) {
            const int* cs = reinterpret_cast<const int*>(smem + warp * kWarpBytes + (i % kStages) * kStageBytes + 2 * kTileBytes);
            lc_lo = fast_log2((float)max(cs[g], 1));
            lc_hi = fast_log2((float)max(cs[g + 8], 1));
        }
        const bool ok_lo = row0 + g < len, ok_hi = row0 + g + 8 < len;
        const float x0 = ok_lo ? fmaf((sa[0] + sb[0]) + (sc2[0] + sd[0]), scale_log2, lc_lo) : -INFINITY;
        const float x1 = ok_lo ? fmaf((sa[1] + sb[1]) + (sc2[1] + sd[1]), scale_log2, lc_lo) : -INFINITY;
        const float x2 = ok_hi ? fmaf((sa[2] + sb[2]) + (sc2[2] + sd[2]), scale_log2, lc_hi) : -INFINITY;
        const float x3 = ok_hi ? fmaf((sa[3] + sb[3]) + (sc2[3] + sd[3]), scale_log2, lc_hi) : -INFINITY;
        // The running maxima m0, m1 are common to the warp.  They are raised only when some lane meets a
        // score more than kMaxSlack above them (one vote per tile instead of a shuffle reduction): the
        // weights 2^(x - m) then stay below 2^kMaxSlack, which fp32 sums and bf16 weights carry without loss.
        const float lx0 = fmaxf(x0, x2), lx1 = fmaxf(x1, x3);
        if (__any_sync(kFull, (lx0 > m0 + kMaxSlack) || (lx1 > m1 + kMaxSlack))) {
            float mx0 = lx0, mx1 = lx1;
#pragma unroll
            for (int off = 4; off < 32; off <<= 1) {
                mx0 = fmaxf(mx0, __shfl_xor_sync(kFull, mx0, off));
                mx1 = fmaxf(mx1, __shfl_xor_sync(kFull, mx1, off));
            }
            const float mn0 = fmaxf(m0, mx0), mn1 = fmaxf(m1, mx1);   // finite: a tile has a valid row
            const float c0 = fast_exp2(m0 - mn0), c1 = fast_exp2(m1 - mn1);
            l0 *= c0; l1 *= c1;
#pragma unroll
            for (int mt = 0; mt < 8; ++mt) { o[mt][0] *= c0; o[mt][2] *= c0; o[mt][1] *= c1; o[mt][3] *= c1; }
            m0 = mn0; m1 = mn1;
        }
        // The weights enter the second product as bf16 pairs (leading part + remainder), which keeps
        // sixteen bits of each: a single bf16 rounding of P would be the largest error of the whole path.
        const float w0 = fast_exp2(x0 - m0), w1 = fast_exp2(x1 - m1);   // row g
        const float w2 = fast_exp2(x2 - m0), w3 = fast_exp2(x3 - m1);   // row g + 8
        const uint32_t p_lo = pack_bf16x2(w0, w1), p_hi = pack_bf16x2(w2, w3);
        const uint32_t r_lo = pack_bf16x2(w0 - bf16_lo(p_lo), w1 - bf16_hi(p_lo));
        const uint32_t r_hi = pack_bf16x2(w2 - bf16_lo(p_hi), w3 - bf16_hi(p_hi));
        l0 += (bf16_lo(p_lo) + bf16_lo(r_lo)) + (bf16_lo(p_hi) + bf16_lo(r_hi));
        l1 += (bf16_hi(p_lo) + bf16_hi(r_lo)) + (bf16_hi(p_hi) + bf16_hi(r_hi));
        const uint32_t pb0 = movmatrix_trans(p_lo), pb1 = movmatrix_trans(p_hi);
        const uint32_t rb0 = movmatrix_trans(r_lo), rb1 = movmatrix_trans(r_hi);

        // O^T += V^T . P^T
#pragma unroll
        for (int mt = 0; mt < 8; ++mt) {
            uint32_t a0, a1, a2, a3;
            const int c = 2 * mt + v_csel;
            ldmatrix_x4_trans(st + kTileBytes + v_row * kRowBytes + ((c ^ (v_row & 7)) << 4), a0, a1, a2, a3);
            mma_bf16(o[mt], a0, a1, a2, a3, pb0, pb1);
            mma_bf16(o[mt], a0, a1, a2, a3, rb0, rb1);
        }
        __syncwarp();
        // the stage just consumed takes the tile three ahead
        const int nxt = i + kStages;
        if (nxt < my_tiles)
            issue_tile(wbase + (i % kStages) * kStageBytes, kh, vh, ch, (t0 + warp + nxt * kWarps) * kTile, len, lane, soff);
        cp_async_commit();
    }
    cp_async_wait<0>();

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
    // ---- block partial (m, l, O) into this block's shared memory, behind the warps' slabs ----
    const float* slabs = reinterpret_cast<const float*>(smem);
    float* blk = reinterpret_cast<float*>(smem) + kWarps * (8 * kD);   // [8][128] O, [8] m, [8] l
    for (int e4 = threadIdx.x; e4 < G * (kD / 4); e4 += kWarps * 32) {
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int w2 = 0; w2 < kWarps; ++w2) {
            const float4 v = *reinterpret_cast<const float4*>(slabs + w2 * (8 * kD) + e4 * 4);
            acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
        }
        *reinterpret_cast<float4*>(blk + e4 * 4) = acc;
    }
    if (threadIdx.x < 8) {
        const int hd = threadIdx.x;
        float bm = -INFINITY, bl = 0.f;
#pragma unroll
        for (int w2 = 0; w2 < kWarps; ++w2) bm = fmaxf(bm, sh_m[w2][hd]);
#pragma unroll
        for (int w2 = 0; w2 < kWarps; ++w2) {
            const float mw = sh_m[w2][hd];
            bl += (mw == -INFINITY) ? 0.f : sh_l[w2][hd] * fast_exp2(mw - bm);
        }
        blk[8 * kD + hd] = bm;
        blk[8 * kD + 8 + hd] = bl;
    }

    // ---- the splits of one thread-block cluster are folded through distributed shared memory ----
    // Every block of the cluster folds its own slice of the (head, column) pairs, reading that slice of
    // every member's partial straight out of the member's shared memory (no trip through L2, no counter,
    // and no single block pulling all partials through its own port); the members stay until all have read.
    cg::cluster_group cluster = cg::this_cluster();
    const int csize = (int)cluster.num_blocks(), crank = (int)cluster.block_rank();
    const int n_clusters = n_split / csize, cidx = split / csize;   // clusters per head, this one's index
    float* my_part = part + ((size_t)bh * n_clusters + cidx) * kPartStride;
    const bool direct = n_clusters == 1;   // this cluster holds the whole head: its fold is the result
    const int n_parts = csize == 1 ? eff_split : n_clusters;   // partials that hold something
    const int slice = (G * (kD / 4) + csize - 1) / csize;
    cluster.sync();
    // Nothing has been written to global memory so far (the block partials live in shared memory).  Under
    // an overlapped launch every global write of this kernel (out, cluster partials, arrival counters) is
    // ordered behind the completion of the kernel before it, which ordered its own writes behind its
    // predecessor in the same way: completion is transitive along a run of overlapped launches, and they
    // may share workspace and out buffers.  (A no-op for an ordinary launch and after the wait above.)
    asm volatile("griddepcontrol.wait;\n" ::: "memory");
    for (int i = threadIdx.x; i < slice; i += kWarps * 32) {
        const int e4 = crank * slice + i;
        if (e4 >= G * (kD / 4)) break;
        const int hd = e4 / (kD / 4), d4 = (e4 % (kD / 4)) * 4;
        float mv[kMaxCluster], lv[kMaxCluster];
        float4 ov[kMaxCluster];
#pragma unroll
        for (int j = 0; j < kMaxCluster; ++j) {
            const float* pb = cluster.map_shared_rank(blk, j < csize ? j : 0);
            mv[j] = j < csize ? pb[8 * kD + hd] : -INFINITY;
            lv[j] = j < csize ? pb[8 * kD + 8 + hd] : 0.f;
            ov[j] = j < csize ? *reinterpret_cast<const float4*>(pb + hd * kD + d4) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
        float gm = mv[0];
#pragma unroll
        for (int j = 1; j < kMaxCluster; ++j) gm = fmaxf(gm, mv[j]);
        float lsum = 0.f;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int j = 0; j < kMaxCluster; ++j) {
            const float w = (mv[j] == -INFINITY) ? 0.f : fast_exp2(mv[j] - gm);
            lsum = fmaf(w, lv[j], lsum);
            acc.x = fmaf(w, ov[j].x, acc.x); acc.y = fmaf(w, ov[j].y, acc.y);
            acc.z = fmaf(w, ov[j].z, acc.z); acc.w = fmaf(w, ov[j].w, acc.w);
        }
        if (direct) {
            const float inv = lsum > 0.f ? 1.f / lsum : 0.f;
            store_out4(out + ((size_t)b * Hq + (size_t)h * G + hd) * kD + d4, acc, inv);
        } else {
            *reinterpret_cast<float4*>(my_part + hd * kD + d4) = acc;
            if (d4 == 0) { my_part[8 * kD + hd] = gm; my_part[8 * kD + 8 + hd] = lsum; }
        }
    }
    if (!direct) __threadfence();   // this block's slice of the cluster partial, before the cluster's ticket
    cluster.sync();   // every member's shared memory has been read: they may leave
    if (direct || crank != 0) return;

    // ---- several partials per head: the last block to arrive merges them ----
    ticket_and_merge(part, tickets, bh, n_clusters, n_parts, G, Hq, b, h, out, &sh_last);
}

// Block split of one head: how many blocks stream it, and how they are grouped into clusters.
struct SplitPlan { int n_split, cluster; };

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

// Splits are grouped into clusters whose blocks fold their partials through distributed shared memory
// when the whole launch is about one wave of blocks (few heads: the latency of the merge is then a large
// part of the launch).  One cluster per head (no partial ever leaves the SMs) whenever the wanted split count is within a
// quarter of the largest cluster; otherwise as few equal clusters as cover it.
inline int rows_per_block(int B, int Hkv, int cap) { return (long long)B * Hkv * cap >= kBigLaunchRows ? kRowsPerBlockBig : kRowsPerBlock; }

inline SplitPlan plan_for(int B, int Hkv, int cap, int sms, int cmax) {
    const int s0 = splits_for(B, Hkv, cap, sms);
    if (s0 <= 1 || cmax <= 1) return {s0, 1};
    // Several waves of blocks (many heads): a block that waits at a cluster barrier holds an SM slot the next
    // wave wants, and the merge is a small part of such a launch; there every block is a cluster of its own,
    // leaves its partial in global memory and goes (measured: clusters of 6 cost 7 % at 128 heads x 8K rows).
    if ((long long)B * Hkv * s0 > 2LL * sms) {
        // ... and the shares are cut finer (a head that is full streams kRowsPerBlock rows per block; how many of
        // the blocks a shorter head uses is settled in the kernel, from its length)
        const int rpb = rows_per_block(B, Hkv, cap);
        const int fine = (cap + rpb - 1) / rpb;
        const int s1 = fine > s0 ? fine : s0;
        return {s1 > 256 ? 256 : s1, 1};
    }
    if (s0 <= cmax + cmax / 4) { const int c = s0 < cmax ? s0 : cmax; return {c, c}; }
    const int k = (s0 + cmax - 1) / cmax, c = s0 / k;
    return {c * k, c};
}

}  // namespace dm

bool decode_mma_supported(const DecodeArgs& a) {
    return a.dt == SC_BF16 && a.d == dm::kD && (a.Hq / a.Hkv) <= 8 && a.cap > 0 && a.Hkv <= 65535 && a.B <= 65535;
}

// Bytes at the front of the workspace that hold the arrival counters (zero between calls).
size_t decode_mma_counter_bytes(int32_t B, int32_t Hkv) { return sizeof(int32_t) * (((size_t)B * Hkv + 63) / 64 * 64); }

size_t decode_mma_ws_bytes(int32_t B, int32_t Hq, int32_t Hkv, int32_t d, int32_t cap) {
    (void)Hq; (void)d;
    // tickets (one per (b, head), zero between calls) + partials for the largest split count
    const int s = dm::plan_for(B, Hkv, cap, 256, dm::kMaxCluster).n_split;
    const int s2 = dm::plan_for(B, Hkv, cap, 132, dm::kMaxCluster).n_split;
    const int s3 = dm::plan_for(B, Hkv, cap, 132, 8).n_split;
    int smax = s > s2 ? s : s2;
    if (s3 > smax) smax = s3;
    const int fine = (cap + dm::kRowsPerBlockBig - 1) / dm::kRowsPerBlockBig;   // the finest split of a launch of several waves
    if (fine > smax) smax = fine > 256 ? 256 : fine;
    return 256 + decode_mma_counter_bytes(B, Hkv) +
           sizeof(float) * (size_t)B * Hkv * smax * dm::kPartStride;
}

cudaError_t launch_decode_mma(const DecodeArgs& a, cudaStream_t st) {
    // per device: SM count, the opt-in to large dynamic shared memory, and the largest cluster that can be scheduled
    static int sms_of[64] = {0}, cmax_of[64] = {0};
    int dev = 0;
    cudaGetDevice(&dev);
    dev &= 63;
    if (sms_of[dev] == 0) {
        int v = 0;
        cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev);
        cudaFuncSetAttribute(dm::decode_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, dm::kSmemBytes);
        int cmax = 8;   // the portable cluster size
        if (cudaFuncSetAttribute(dm::decode_mma_kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess) {
            cudaLaunchConfig_t probe = {};
            probe.gridDim = dim3(dm::kMaxCluster, 1, 1);
            probe.blockDim = dim3(dm::kWarps * 32);
            probe.dynamicSmemBytes = dm::kSmemBytes;
            cudaLaunchAttribute pa[1];
            pa[0].id = cudaLaunchAttributeClusterDimension;
            pa[0].val.clusterDim.x = dm::kMaxCluster; pa[0].val.clusterDim.y = 1; pa[0].val.clusterDim.z = 1;
            probe.attrs = pa;
            probe.numAttrs = 1;
            int n_clusters = 0;
            if (cudaOccupancyMaxActiveClusters(&n_clusters, dm::decode_mma_kernel, &probe) == cudaSuccess && n_clusters > 0)
                cmax = dm::kMaxCluster;
        }
        (void)cudaGetLastError();   // a refused opt-in or probe is not an error of this call
        cmax_of[dev] = cmax;
        sms_of[dev] = v > 256 ? 256 : (v < 1 ? 1 : v);
    }
    const dm::SplitPlan plan = dm::plan_for(a.B, a.Hkv, a.cap, sms_of[dev], cmax_of[dev]);
    int32_t* tickets = (int32_t*)a.ws;
    float* part = (float*)((char*)a.ws + decode_mma_counter_bytes(a.B, a.Hkv));
    const float scale = (a.scale == 0.f ? 1.f / sqrtf((float)a.d) : a.scale) * 1.4426950408889634f;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(plan.n_split, a.Hkv, a.B);
    cfg.blockDim = dim3(dm::kWarps * 32);
    cfg.dynamicSmemBytes = dm::kSmemBytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = plan.cluster; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = (a.flags & (SC_FLAG_OVERLAP_PREV | SC_FLAG_OVERLAP_CHAIN)) ? 2 : 1;
    const int q_from_prev = (a.flags & SC_FLAG_OVERLAP_CHAIN) ? 1 : 0;
    // fewest blocks a head is shared out among, however short it is: three blocks per SM over the launch
    const int heads = a.B * a.Hkv;
    const int min_split = (3 * sms_of[dev] + heads - 1) / heads;
    note_launches(1);
    return cudaLaunchKernelEx(&cfg, dm::decode_mma_kernel, (const __nv_bfloat16*)a.q, a.Hq, a.Hkv,
                              (const __nv_bfloat16*)a.core_k, (const __nv_bfloat16*)a.core_v, a.count, a.cap,
                              a.core_len, scale, plan.n_split, min_split, dm::rows_per_block(a.B, a.Hkv, a.cap), q_from_prev, (__nv_bfloat16*)a.out, part, tickets);
}

}  // namespace sc
