// Fused bf16 compress kernel (d = 128, token stride of 256 bytes or more), sm_100a.
//
// One block per (sequence, KV head, work tile).  A tile is a run of whole segments of at most
// SC_TILE_ROWS tokens (K and V staged in shared memory), or one longer segment alone (K staged,
// V streamed from global memory).  Steps inside a block:
//   1. cp.async the tile's K (and V) rows into shared memory, 16-byte chunks XOR-swizzled;
//   2. Gram blocks K.K^T of 32x32 rows on the tensor cores (mma.m16n8k16, bf16 products are exact
//      in fp32) for exactly the block pairs a segment spans; the diagonal gives the norms, then
//      Sim > tau (Eq. 2) is decided as G_ij > tau*|k_i|*|k_j| and packed into one adjacency bit
//      row per token (later tokens of the same segment only);
//   3. Algorithm 1 per segment on those bit rows: lowest unassigned token becomes a seed and
//      takes every unassigned adjacent token -- a few word operations per seed, one warp per
//      segment with one lane per 32-token word;
//   4. the tile's cluster count feeds a prefix sum over the tiles of the (sequence, head): either
//      a separate count pass (two-pass mode) or a decoupled look-back over per-tile status words
//      (single pass; tiles are taken in ticket order so every predecessor is already running,
//      and the wait is bounded);
//   5. Eq. 3: one warp per cluster sums the member rows of K and V in token order in fp32,
//      scales by 1/|S|, rounds once to bf16 and writes the core row and its count compactly.
#include "common.cuh"

namespace sc {

namespace cf {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kD = 128;
constexpr int kRowBytes = 256;
constexpr int kMaxRows = SC_MAX_CHUNK_LEN;        // 256: a long tile
constexpr int kShortRows = SC_TILE_ROWS;          // 128
constexpr int kNW = 8;                            // 32-bit words per adjacency row
constexpr int kKvBytes = kMaxRows * kRowBytes;    // 65536: short = K 32K | V 32K, long = K 64K
constexpr int kAdjOff = kKvBytes;
constexpr int kAdjBytes = kMaxRows * kNW * 4;     // 8192
constexpr int kNormOff = kAdjOff + kAdjBytes;     // float[256]
constexpr int kSendOff = kNormOff + kMaxRows * 4; // uint16[256]: segment end per row
constexpr int kSegsOff = kSendOff + kMaxRows * 2; // int16[130]: segment starts in the tile
constexpr int kItemOff = kSegsOff + 272;          // uint8[48]: (row block << 4 | col block) pairs
constexpr int kMiscOff = kItemOff + 48;           // uint32 seedmask[8], int misc[8]
constexpr int kSmemBytes = kMiscOff + 64;

enum Mode { kCountOnly = 0, kWriteWithCounts = 1, kLookBack = 2 };

constexpr uint32_t kFlagAggregate = 1u << 30, kFlagPrefix = 2u << 30, kValueMask = (1u << 30) - 1;
constexpr int kSpinLimit = 1 << 22;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory"); }
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t swz(int row, int chunk) { return row * kRowBytes + ((chunk ^ (row & 7)) << 4); }
__device__ __forceinline__ uint32_t bits_between(int lo, int hi, int word) {   // bits [lo, hi) that fall in `word`
    lo = max(lo, word * 32); hi = min(hi, word * 32 + 32);
    if (hi <= lo) return 0u;
    return (0xffffffffu >> (32 - (hi - lo))) << (lo - word * 32);
}
__device__ __forceinline__ uint32_t ld_volatile(const uint32_t* p) {
    uint32_t v;
    asm volatile("ld.volatile.global.u32 %0, [%1];\n" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// 32x32 block of K.K^T: rows of block rb against rows of block cb.
__device__ __forceinline__ void gram_block(uint32_t kbase, int rb, int cb, int lane, float (&acc)[2][4][4]) {
#pragma unroll
    for (int mt = 0; mt < 2; ++mt)
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) acc[mt][nt][0] = acc[mt][nt][1] = acc[mt][nt][2] = acc[mt][nt][3] = 0.f;
    const int j = lane >> 3, r8 = lane & 7;
    const int a_row = r8 + ((j & 1) << 3), a_c = j >> 1;      // (r0-7,c) (r8-15,c) (r0-7,c+1) (r8-15,c+1)
    const int b_row = r8 + ((j >> 1) << 3), b_c = j & 1;      // (r0-7,c) (r0-7,c+1) (r8-15,c) (r8-15,c+1)
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
        uint32_t a[2][4], bq[2][4];
#pragma unroll
        for (int mt = 0; mt < 2; ++mt) {
            const int row = rb * 32 + mt * 16 + a_row;
            ldmatrix_x4(kbase + swz(row, 2 * ks + a_c), a[mt][0], a[mt][1], a[mt][2], a[mt][3]);
        }
#pragma unroll
        for (int p = 0; p < 2; ++p) {
            const int row = cb * 32 + p * 16 + b_row;
            ldmatrix_x4(kbase + swz(row, 2 * ks + b_c), bq[p][0], bq[p][1], bq[p][2], bq[p][3]);
        }
#pragma unroll
        for (int mt = 0; mt < 2; ++mt)
#pragma unroll
            for (int nt = 0; nt < 4; ++nt)
                mma_bf16(acc[mt][nt], a[mt][0], a[mt][1], a[mt][2], a[mt][3], bq[nt >> 1][(nt & 1) * 2], bq[nt >> 1][(nt & 1) * 2 + 1]);
    }
}

// Turns a Gram block into adjacency words: bit j of adj[i][cb] = Sim(i, 32cb + j) > tau, limited
// to later tokens of i's own segment.
__device__ __forceinline__ void threshold_block(const float (&acc)[2][4][4], int rb, int cb, int lane, float tau,
                                                const float* norm, const uint16_t* send, uint32_t* adj) {
    const int g = lane >> 2, tig = lane & 3;
    float tn[4][2];
#pragma unroll
    for (int nt = 0; nt < 4; ++nt) {
        tn[nt][0] = tau * norm[cb * 32 + nt * 8 + 2 * tig];
        tn[nt][1] = tau * norm[cb * 32 + nt * 8 + 2 * tig + 1];
    }
#pragma unroll
    for (int mt = 0; mt < 2; ++mt)
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
            const int i = rb * 32 + mt * 16 + hh * 8 + g;
            const float ni = norm[i];
            uint32_t w = 0;
#pragma unroll
            for (int nt = 0; nt < 4; ++nt)
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const float thr = ni * tn[nt][e];
                    bool hit = acc[mt][nt][hh * 2 + e] > thr;
                    if (tau < 0.f) hit = hit || (thr == 0.f);   // a zero-norm key has Sim = 0 > tau
                    w |= (hit ? 1u : 0u) << (nt * 8 + 2 * tig + e);
                }
            w |= __shfl_xor_sync(kFull, w, 1);
            w |= __shfl_xor_sync(kFull, w, 2);
            if (tig == 0) adj[i * kNW + cb] = w & bits_between(i + 1, (int)send[i], cb);
        }
}

template <int kMode>
__global__ void __launch_bounds__(kThreads, 3)
compress_fused_kernel(const __nv_bfloat16* __restrict__ K, const __nv_bfloat16* __restrict__ V, sc_strides st,
                      int Hkv, int n, const int32_t* __restrict__ seg_off, const int32_t* __restrict__ tile_seg,
                      const int32_t* __restrict__ seq_tile_cnt, int n_tile_cap, float tau,
                      __nv_bfloat16* __restrict__ core_k, __nv_bfloat16* __restrict__ core_v,
                      int32_t* __restrict__ count, int cap, int32_t* __restrict__ core_len,
                      int32_t* __restrict__ assign, uint32_t* __restrict__ tile_state, int32_t* __restrict__ tickets,
                      int32_t* status) {
    extern __shared__ __align__(128) unsigned char smem[];
    uint32_t* adj = reinterpret_cast<uint32_t*>(smem + kAdjOff);
    float* norm = reinterpret_cast<float*>(smem + kNormOff);
    uint16_t* send = reinterpret_cast<uint16_t*>(smem + kSendOff);
    int16_t* segs = reinterpret_cast<int16_t*>(smem + kSegsOff);
    uint8_t* items = reinterpret_cast<uint8_t*>(smem + kItemOff);
    uint32_t* seedmask = reinterpret_cast<uint32_t*>(smem + kMiscOff);
    int* misc = reinterpret_cast<int*>(smem + kMiscOff + 32);   // [0] tile index, [1] n items, [2] base offset

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int h = blockIdx.y, b = blockIdx.z;
    const int bh = b * Hkv + h;
    const int n_tiles = min(seq_tile_cnt[b], n_tile_cap);

    // ---- which tile ----
    int t;
    if (kMode == kLookBack) {   // ticket order: every earlier tile of this head is held by a running block
        if (tid == 0) misc[0] = atomicAdd(&tickets[bh], 1);
        __syncthreads();
        t = misc[0];
    } else {
        t = blockIdx.x;
    }
    if (t >= n_tiles) return;

    const int32_t* ts = tile_seg + (size_t)b * (n_tile_cap + 1);
    const int s_begin = ts[t], s_end = ts[t + 1];
    const int nseg = min(s_end - s_begin, kShortRows);
    const int g_row0 = seg_off[s_begin];                       // on the flattened [B*n] axis
    const int R = min(seg_off[s_begin + nseg] - g_row0, kMaxRows);
    const int row0 = g_row0 - b * n;                           // within the sequence
    const bool long_tile = R > kShortRows;
    const int nrb = (R + 31) >> 5;

    // ---- 1. stage K (and V) ----
    const uint32_t sbase = smem_u32(smem);
    const __nv_bfloat16* Kt = K + b * st.b + h * st.h + (int64_t)row0 * st.n;
    const __nv_bfloat16* Vt = V + b * st.b + h * st.h + (int64_t)row0 * st.n;
    {
        const int c = tid & 15;
        for (int r = tid >> 4; r < R; r += kThreads / 16) cp_async16(sbase + swz(r, c), Kt + (int64_t)r * st.n + c * 8);
        cp_async_commit();
        if (kMode != kCountOnly && !long_tile)
            for (int r = tid >> 4; r < R; r += kThreads / 16)
                cp_async16(sbase + kShortRows * kRowBytes + swz(r, c), Vt + (int64_t)r * st.n + c * 8);
        cp_async_commit();
    }

    // ---- segment bookkeeping (while the copies fly) ----
    for (int i = tid; i <= nseg; i += kThreads) segs[i] = (int16_t)min(seg_off[s_begin + i] - g_row0, kMaxRows);
    if (tid < kNW) seedmask[tid] = 0u;
    __syncthreads();
    for (int r = tid; r < nrb * 32; r += kThreads) {   // end of the segment each row belongs to (0 past the tile)
        int lo = 0, hi = nseg;                         // find s with segs[s] <= r < segs[s+1]
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (segs[mid] <= r) lo = mid; else hi = mid;
        }
        send[r] = (r < R) ? (uint16_t)segs[lo + 1] : (uint16_t)0;
    }
    __syncthreads();
    if (tid == 0) {   // list the Gram blocks: diagonals first, then the blocks right of them a segment reaches
        int k = 0;
        for (int rb = 0; rb < nrb; ++rb) items[k++] = (uint8_t)((rb << 4) | rb);
        for (int rb = 0; rb < nrb; ++rb) {
            const int last = min(rb * 32 + 31, R - 1);
            const int cbmax = ((int)send[last] - 1) >> 5;
            for (int cb = rb + 1; cb <= cbmax; ++cb) items[k++] = (uint8_t)((rb << 4) | cb);
        }
        misc[1] = k;
    }
    cp_async_wait<1>();   // K has landed (this thread's copies); the barrier publishes everyone's
    __syncthreads();

    // ---- 2. Gram blocks -> norms -> adjacency bits ----
    const int n_items = misc[1];
    {
        float acc[2][4][4];
        const bool have = warp < n_items;
        int rb = 0, cb = 0;
        if (have) {
            rb = items[warp] >> 4; cb = items[warp] & 15;
            gram_block(sbase, rb, cb, lane, acc);
            if (rb == cb) {   // diagonal of the Gram block = squared norms
                const int g = lane >> 2, tig = lane & 3;
                if ((g >> 1) == tig) {
                    const int e = g & 1;
#pragma unroll
                    for (int mt = 0; mt < 2; ++mt)
#pragma unroll
                        for (int hh = 0; hh < 2; ++hh)
                            norm[rb * 32 + mt * 16 + hh * 8 + g] =
                                sqrtf(e ? acc[mt][2 * mt + hh][hh * 2 + 1] : acc[mt][2 * mt + hh][hh * 2]);
                }
            }
        }
        __syncthreads();
        if (have) threshold_block(acc, rb, cb, lane, tau, norm, send, adj);
        for (int k = warp + kWarps; k < n_items; k += kWarps) {
            rb = items[k] >> 4; cb = items[k] & 15;
            gram_block(sbase, rb, cb, lane, acc);
            threshold_block(acc, rb, cb, lane, tau, norm, send, adj);
        }
    }
    __syncthreads();

    // ---- 3. Algorithm 1 per segment: one warp per segment, lane c owns word c ----
    int32_t* as = assign ? assign + (size_t)bh * n + row0 : nullptr;
    for (int s = warp; s < nseg; s += kWarps) {
        const int a = segs[s], e = segs[s + 1];
        if (e - a == 1) {   // a delimiter or a one-token run: its own cluster
            if (lane == 0) {
                adj[a * kNW + (a >> 5)] = 1u << (a & 31);
                atomicOr(&seedmask[a >> 5], 1u << (a & 31));
                if (as) as[a] = row0 + a;
            }
            continue;
        }
        const int w0 = a >> 5, w1 = (e - 1) >> 5;
        uint32_t U = (lane < kNW) ? bits_between(a, e, lane) : 0u;   // unassigned tokens of this segment
        uint32_t seeds = 0u;
        for (;;) {
            const uint32_t any = __ballot_sync(kFull, U != 0u);
            if (any == 0u) break;
            const int wf = __ffs(any) - 1;
            const int i = wf * 32 + __ffs(__shfl_sync(kFull, U, wf)) - 1;   // lowest unassigned token: a seed
            uint32_t mem = 0u;
            if (lane >= w0 && lane <= w1) {
                mem = adj[i * kNW + lane] & U;
                if (lane == wf) { mem |= 1u << (i & 31); seeds |= 1u << (i & 31); }
                adj[i * kNW + lane] = mem;            // the row now lists the cluster's members
                U &= ~mem;
                if (as) {
                    uint32_t mm = mem;
                    while (mm) { const int j = lane * 32 + __ffs(mm) - 1; mm &= mm - 1; as[j] = row0 + i; }
                }
            }
        }
        if (seeds) atomicOr(&seedmask[lane], seeds);
    }
    __syncthreads();

    // ---- 4. output offset of this tile ----
    int P = 0;
#pragma unroll
    for (int w = 0; w < kNW; ++w) P += __popc(seedmask[w]);
    if (kMode == kCountOnly) {
        if (tid == 0) tile_state[(size_t)bh * n_tile_cap + t] = (uint32_t)P;
        return;
    }
    if (warp == 0) {
        int base = 0;
        uint32_t* stt = tile_state + (size_t)bh * n_tile_cap;
        if (kMode == kWriteWithCounts) {
            for (int k = lane; k < t; k += 32) base += (int)stt[k];
            base = warp_sum_i(base);
        } else {
            if (lane == 0) atomicExch(&stt[t], (t == 0 ? kFlagPrefix : kFlagAggregate) | (uint32_t)P);
            // look back over the predecessors, 32 at a time, nearest first
            int upto = t;      // tiles [0, upto) still to be accounted for
            int spins = 0;
            bool gave_up = false;
            while (upto > 0) {
                const int k = upto - 1 - lane;
                uint32_t v = (k >= 0) ? ld_volatile(&stt[k]) : kFlagPrefix;   // before tile 0: prefix 0
                const uint32_t ready = __ballot_sync(kFull, (v >> 30) != 0u);
                const uint32_t pref = __ballot_sync(kFull, (v >> 30) == 2u);
                // usable run: lanes 0..m-1 all ready, stopping at the first that holds a full prefix
                const int first_unready = (ready == kFull) ? 32 : __ffs(~ready) - 1;
                const int first_pref = pref ? __ffs(pref) - 1 : 32;
                const int take = min(first_unready, first_pref + 1);
                int contrib = (lane < take) ? (int)(v & kValueMask) : 0;
                base += warp_sum_i(contrib);
                if (first_pref < first_unready) break;        // reached an inclusive prefix
                upto -= take;
                if (take == 0) {
                    if (++spins > kSpinLimit) { gave_up = true; break; }
                    __nanosleep(40);
                }
            }
            if (gave_up) { set_status(status, SC_ERR_TIMEOUT); base = 0; }
            if (lane == 0 && t > 0) atomicExch(&stt[t], kFlagPrefix | (uint32_t)(base + P));
        }
        if (lane == 0) {
            misc[2] = base;
            if (t == n_tiles - 1) {
                core_len[bh] = base + P;
                if (base + P > cap) set_status(status, SC_ERR_CAPACITY);
            }
        }
    }
    cp_async_wait<0>();   // V
    __syncthreads();
    const int base = misc[2];

    // ---- 5. Eq. 3: one warp per cluster ----
    const unsigned char* ksm = smem;
    const unsigned char* vsm = smem + kShortRows * kRowBytes;
    const size_t obase = (size_t)bh * cap;
    int rank_base = 0;
    for (int w = 0; w < nrb; ++w) {
        const uint32_t sm = seedmask[w];
        uint32_t m = sm;
        while (m) {
            const int bit = __ffs(m) - 1;
            m &= m - 1;
            const int rank = rank_base + __popc(sm & ((1u << bit) - 1u));
            if ((rank & (kWarps - 1)) != warp) continue;
            const int i = w * 32 + bit;
            const int w1 = ((int)send[i] - 1) >> 5;
            float ak[4] = {0.f, 0.f, 0.f, 0.f}, av[4] = {0.f, 0.f, 0.f, 0.f};
            int cnt = 0;
            for (int ww = w; ww <= w1; ++ww) {
                uint32_t mm = adj[i * kNW + ww];
                cnt += __popc(mm);
                while (mm) {
                    const int j = ww * 32 + __ffs(mm) - 1;
                    mm &= mm - 1;
                    const uint32_t off = swz(j, lane >> 1) + (lane & 1) * 8;
                    const uint2 kk = *reinterpret_cast<const uint2*>(ksm + off);
                    uint2 vv;
                    if (!long_tile) vv = *reinterpret_cast<const uint2*>(vsm + off);
                    else vv = __ldg(reinterpret_cast<const uint2*>(Vt + (int64_t)j * st.n + lane * 4));
                    ak[0] += __uint_as_float(kk.x << 16); ak[1] += __uint_as_float(kk.x & 0xffff0000u);
                    ak[2] += __uint_as_float(kk.y << 16); ak[3] += __uint_as_float(kk.y & 0xffff0000u);
                    av[0] += __uint_as_float(vv.x << 16); av[1] += __uint_as_float(vv.x & 0xffff0000u);
                    av[2] += __uint_as_float(vv.y << 16); av[3] += __uint_as_float(vv.y & 0xffff0000u);
                }
            }
            const int row = base + rank;
            if (row < cap) {
                const float inv = 1.0f / (float)cnt;
                __nv_bfloat162 k01 = __floats2bfloat162_rn(ak[0] * inv, ak[1] * inv);
                __nv_bfloat162 k23 = __floats2bfloat162_rn(ak[2] * inv, ak[3] * inv);
                __nv_bfloat162 v01 = __floats2bfloat162_rn(av[0] * inv, av[1] * inv);
                __nv_bfloat162 v23 = __floats2bfloat162_rn(av[2] * inv, av[3] * inv);
                uint2 ko, vo;
                ko.x = *reinterpret_cast<uint32_t*>(&k01); ko.y = *reinterpret_cast<uint32_t*>(&k23);
                vo.x = *reinterpret_cast<uint32_t*>(&v01); vo.y = *reinterpret_cast<uint32_t*>(&v23);
                *reinterpret_cast<uint2*>(core_k + (obase + row) * kD + lane * 4) = ko;
                *reinterpret_cast<uint2*>(core_v + (obase + row) * kD + lane * 4) = vo;
                if (lane == 0) count[obase + row] = cnt;
            }
        }
        rank_base += __popc(sm);
    }
}

}  // namespace cf

bool compress_fused_supported(const CompressArgs& a) {
    return a.dt == SC_BF16 && a.d == cf::kD && a.Hkv <= 65535 && a.B <= 65535 && a.n_tile_cap >= 1;
}

size_t compress_fused_ws_bytes(int32_t B, int32_t Hkv, int32_t n) {
    const size_t tiles = 2 * (size_t)div_up(n, SC_TILE_ROWS) + 1;
    return sizeof(uint32_t) * (size_t)B * Hkv * (tiles + 1) + 256;
}

cudaError_t launch_compress_fused(const CompressArgs& a, cudaStream_t st) {
    static bool attr_set[64] = {false};
    int dev = 0;
    cudaGetDevice(&dev);
    dev &= 63;
    if (!attr_set[dev]) {
        cudaFuncSetAttribute(cf::compress_fused_kernel<cf::kCountOnly>, cudaFuncAttributeMaxDynamicSharedMemorySize, cf::kSmemBytes);
        cudaFuncSetAttribute(cf::compress_fused_kernel<cf::kWriteWithCounts>, cudaFuncAttributeMaxDynamicSharedMemorySize, cf::kSmemBytes);
        cudaFuncSetAttribute(cf::compress_fused_kernel<cf::kLookBack>, cudaFuncAttributeMaxDynamicSharedMemorySize, cf::kSmemBytes);
        attr_set[dev] = true;
    }
    const size_t heads = (size_t)a.B * a.Hkv;
    uint32_t* tile_state = (uint32_t*)a.ws;
    int32_t* tickets = (int32_t*)(tile_state + heads * a.n_tile_cap);
    dim3 grid(a.n_tile_cap, a.Hkv, a.B);
    const __nv_bfloat16* K = (const __nv_bfloat16*)a.K;
    const __nv_bfloat16* V = (const __nv_bfloat16*)a.V;
    __nv_bfloat16* ck = (__nv_bfloat16*)a.core_k;
    __nv_bfloat16* cv = (__nv_bfloat16*)a.core_v;
    if (a.flags & SC_FLAG_TWO_PASS) {
        cf::compress_fused_kernel<cf::kCountOnly><<<grid, cf::kThreads, cf::kSmemBytes, st>>>(
            K, V, a.st, a.Hkv, a.n, a.seg_off, a.tile_seg, a.seq_tile_cnt, a.n_tile_cap, a.tau, ck, cv, a.count, a.cap,
            a.core_len, nullptr, tile_state, tickets, a.status);
        cf::compress_fused_kernel<cf::kWriteWithCounts><<<grid, cf::kThreads, cf::kSmemBytes, st>>>(
            K, V, a.st, a.Hkv, a.n, a.seg_off, a.tile_seg, a.seq_tile_cnt, a.n_tile_cap, a.tau, ck, cv, a.count, a.cap,
            a.core_len, a.assign, tile_state, tickets, a.status);
        note_launches(2);
    } else {
        cudaError_t e = cudaMemsetAsync(a.ws, 0, sizeof(uint32_t) * heads * (a.n_tile_cap + 1), st);
        if (e != cudaSuccess) return e;
        cf::compress_fused_kernel<cf::kLookBack><<<grid, cf::kThreads, cf::kSmemBytes, st>>>(
            K, V, a.st, a.Hkv, a.n, a.seg_off, a.tile_seg, a.seq_tile_cnt, a.n_tile_cap, a.tau, ck, cv, a.count, a.cap,
            a.core_len, a.assign, tile_state, tickets, a.status);
        note_launches(1);
    }
    return cudaGetLastError();
}

}  // namespace sc
