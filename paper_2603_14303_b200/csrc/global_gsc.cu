// Global clustering without chunking: the "none/global" arm of the paper's chunking ablation (Table 4a),
// i.e. Algorithm 1 (Sec. 2.3) with each whole sequence as one chunk, then Eq. 3 (Sec. 2.4).
//
// Algorithm 1 over one long chunk is a sequential greedy pass, but its result has a closed form: the
// seeds are the lexicographically first maximal independent set of the graph {Sim(k_i, k_j) > tau}, and
// every other token joins its lowest adjacent seed.  That is computed here in parallel:
//   1. norms of all keys;
//   2. the adjacency bits of every pair j < i, one 128 x 128 tile of K.K^T at a time on the tensor
//      cores (tcgen05.mma, operands staged by TMA in 128-byte-swizzled shared memory, accumulators in
//      tensor memory, double-buffered so that thresholding tile t overlaps the product of tile t+1),
//      thresholded as G_ij > tau * |k_i| * |k_j| and packed to one bit per pair in a lower-triangular
//      store; a CUDA-core version serves other dtypes and head sizes;
//   3. decision rounds: a token with no undecided earlier neighbour becomes a seed if all its earlier
//      neighbours are members, a token with an earlier neighbour that is a seed becomes a member.  Both
//      rules only ever state final facts, so the fixed point is Algorithm 1's result whatever the
//      order of evaluation; the lowest undecided token is always decidable, so it is reached.  A fixed
//      number of rounds is enqueued (clustered keys need three or four); rounds that find nothing left
//      return at once, and a last kernel finishes whatever is left one head per block;
//   4. every member's seed (its lowest adjacent seed), the seeds' ranks (prefix sum) and core_len;
//   5. Eq. 3: the tokens are binned by cluster (sizes, prefix sum, fill), then one warp per cluster puts
//      its members in token order and sums them (fp32), divides once, rounds once.
#include "common.cuh"
#include "umma.cuh"

namespace sc {

namespace gl {

using namespace umma;

constexpr int kT = 128;                 // tokens per tile side
constexpr int kJChunk = 16;             // column tiles one block walks
constexpr int kHalfBytes = kT * 128;    // one column half (64 bf16) of a staged tile
constexpr int kTileBytes = 2 * kHalfBytes;
constexpr int kThreads = 192;           // warp 0: TMA, warp 1: MMA + tensor memory, warps 2-5: thresholding
constexpr int kTmemCols = 256;          // two 128-column accumulators
constexpr int kSmemA = 0, kSmemB = kTileBytes, kSmemNrm = 3 * kTileBytes, kSmemBar = kSmemNrm + 2 * kT * 4;
constexpr int kSmemBytes = kSmemBar + 128 + 1024;   // + slack to align the base to 1024 bytes
constexpr int kRounds = 12;             // decision rounds enqueued before the finishing kernel

__host__ __device__ inline size_t tile_row_base(size_t I) { return 256 * I * (I + 1); }   // words before tile row I
__host__ __device__ inline size_t bits_words(size_t nb) { return 256 * nb * (nb + 1); }   // per (sequence, head)

struct AdjParams {
    CUtensorMap map;        // keys, boxes of 128 rows x 64 columns
    const float* norms;     // [B*Hkv, n]
    uint32_t* bits;         // [B*Hkv][bits_words(nb)]
    int n, nb, Hkv;
    float tau;
    int32_t* status;
};

template <typename T>
__global__ void __launch_bounds__(256) norms_kernel(const T* __restrict__ K, sc_strides st, int Hkv, int n, int d,
                                                    long long rows, float* __restrict__ norms) {
    const int lane = threadIdx.x & 31;
    const long long row = (long long)blockIdx.x * 8 + (threadIdx.x >> 5);
    if (row >= rows) return;
    const long long bh = row / n, t = row - bh * n;
    const T* kr = K + (bh / Hkv) * st.b + (bh % Hkv) * st.h + t * st.n;
    float acc = 0.f;
    for (int c = lane; c < d; c += 32) { const float x = Elem<T>::load(kr + c); acc = fmaf(x, x, acc); }
    acc = warp_sum(acc);
    if (lane == 0) norms[row] = sqrtf(acc);
}

// Step 2 on the tensor cores: block (I, chunk, head) thresholds tiles (I, J) for J in its chunk, J <= I.
template <bool kNegTau>   // tau < 0: a zero-norm key (Sim = 0) counts as similar
__global__ void __launch_bounds__(kThreads, 2) adj_umma_kernel(const __grid_constant__ AdjParams p) {
    extern __shared__ unsigned char smem_raw[];
    const int I = blockIdx.x, j_begin = blockIdx.y * kJChunk, bh = blockIdx.z;
    if (j_begin > I) return;
    const int nt = min(kJChunk, I + 1 - j_begin);
    const int b = bh / p.Hkv, h = bh % p.Hkv;
    const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;   // the swizzle pattern repeats every 1024 bytes
    unsigned char* smem = smem_raw + (sbase - smem_u32(smem_raw));
    float* nrm_s = reinterpret_cast<float*>(smem + kSmemNrm);      // [2][128]
    const uint32_t bar0 = sbase + kSmemBar;
    const uint32_t a_full = bar0, full0 = bar0 + 8, empty0 = bar0 + 24, tfull0 = bar0 + 40, tempty0 = bar0 + 56;
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + kSmemBar + 72);
    volatile int* sh_fail = reinterpret_cast<volatile int*>(smem + kSmemBar + 76);
    volatile int* sh_issued = reinterpret_cast<volatile int*>(smem + kSmemBar + 80);   // tiles whose loads were issued
    volatile int* sh_fail_thr = reinterpret_cast<volatile int*>(smem + kSmemBar + 84); // set by the thresholding warps only

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        mbar_init(a_full, 1);
        for (int s = 0; s < 2; ++s) {
            mbar_init(full0 + 8 * s, 1);
            mbar_init(empty0 + 8 * s, 1);
            mbar_init(tfull0 + 8 * s, 1);
            mbar_init(tempty0 + 8 * s, 4);
        }
        mbar_fence_init();
        *sh_fail = 0;
        *sh_issued = 0;
        *sh_fail_thr = 0;
    }
    if (warp == 1) tmem_alloc(sbase + kSmemBar + 72, kTmemCols);
    fence_before_sync();
    __syncthreads();
    fence_after_sync();
    const uint32_t tmem = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {   // ---- TMA producer ----
            mbar_expect_tx(a_full, kTileBytes);
            tma_load_4d(sbase + kSmemA, &p.map, 0, I * kT, h, b, a_full);
            tma_load_4d(sbase + kSmemA + kHalfBytes, &p.map, 64, I * kT, h, b, a_full);
            for (int t = 0; t < nt; ++t) {
                const int s = t & 1;
                if (t >= 2 && !mbar_wait(empty0 + 8 * s, ((t >> 1) - 1) & 1)) { *sh_fail = 1; break; }
                const uint32_t dst = sbase + kSmemB + s * kTileBytes;
                mbar_expect_tx(full0 + 8 * s, kTileBytes);
                tma_load_4d(dst, &p.map, 0, (j_begin + t) * kT, h, b, full0 + 8 * s);
                tma_load_4d(dst + kHalfBytes, &p.map, 64, (j_begin + t) * kT, h, b, full0 + 8 * s);
                *sh_issued = t + 1;
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {   // ---- MMA issuer ----
            constexpr uint32_t idesc = instr_desc_bf16(kT, kT, false, false);
            bool ok = mbar_wait(a_full, 0);
            for (int t = 0; t < nt && ok; ++t) {
                const int s = t & 1;
                ok = mbar_wait(full0 + 8 * s, (t >> 1) & 1);
                if (ok && t >= 2) ok = mbar_wait(tempty0 + 8 * s, ((t >> 1) - 1) & 1);
                if (!ok) break;
                fence_after_sync();
                const uint32_t a = sbase + kSmemA, bq = sbase + kSmemB + s * kTileBytes;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {   // sixteen columns of the contraction per instruction
                    const uint32_t off = (ks >> 2) * kHalfBytes + (ks & 3) * 32;
                    mma_bf16_ss(tmem + s * kT, smem_desc_sw128(a + off, 16, 1024), smem_desc_sw128(bq + off, 16, 1024), idesc, ks > 0);
                }
                mma_commit(empty0 + 8 * s);    // the staged tile may be overwritten
                mma_commit(tfull0 + 8 * s);    // the accumulator may be read
            }
            if (!ok) *sh_fail = 1;
        }
    } else {
        // ---- thresholding: thread = one row of the tile (tensor-memory lane), 128 columns per tile ----
        const int q = warp & 3, r = q * 32 + lane;          // warps 2..5 own lane quarters 2, 3, 0, 1
        const int i = I * kT + r;
        const float ni = i < p.n ? p.norms[(size_t)bh * p.n + i] : 0.f;
        uint32_t* row = p.bits + (size_t)bh * bits_words(p.nb) + tile_row_base(I) + (size_t)r * 4 * (I + 1);
        for (int t = 0; t < nt; ++t) {
            const int s = t & 1, J = j_begin + t;
            const int jt = J * kT + r;
            nrm_s[s * kT + r] = jt < p.n ? p.tau * p.norms[(size_t)bh * p.n + jt] : 0.f;
            if (!mbar_wait(tfull0 + 8 * s, (t >> 1) & 1)) { *sh_fail = 1; *sh_fail_thr = 1; }
            fence_after_sync();
            asm volatile("bar.sync 1, 128;\n" ::: "memory");   // the four thresholding warps: column norms are in place
            if (*sh_fail_thr) break;                            // a wait gave up: all four warps leave together
            uint32_t words[4];
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t g[32];
                tmem_ld32(tmem + ((uint32_t)(q * 32) << 16) + s * kT + c * 32, g);
                tmem_ld_wait();
                uint32_t w = 0;
#pragma unroll
                for (int k = 0; k < 32; ++k) {
                    const float thr = ni * nrm_s[s * kT + c * 32 + k];
                    bool hit = __uint_as_float(g[k]) > thr;
                    if (kNegTau) hit = hit || (thr == 0.f);   // a zero-norm key has Sim = 0 > tau
                    w |= (hit ? 1u : 0u) << k;
                }
                if (J == I) {   // earlier tokens only
                    const int keep = r - c * 32;
                    w &= keep >= 32 ? 0xffffffffu : (keep <= 0 ? 0u : ((1u << keep) - 1u));
                }
                words[c] = w;
            }
            fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(tempty0 + 8 * s);
            if (i < p.n) *reinterpret_cast<uint4*>(row + 4 * J) = make_uint4(words[0], words[1], words[2], words[3]);
        }
    }
    __syncthreads();
    if (*sh_fail) {   // a wait gave up: report it and give copies still in flight one more bounded wait
        if (tid == 0) {
            set_status(p.status, SC_ERR_TIMEOUT);
            const int issued = *sh_issued;
            mbar_wait(a_full, 0);
            for (int t = max(issued - 2, 0); t < issued; ++t) mbar_wait(full0 + 8 * (t & 1), (t >> 1) & 1);
        }
        __syncthreads();
    }
    fence_before_sync();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, kTmemCols);
}

// Step 2 on the CUDA cores (any dtype, any d): same grid, same bit layout.
template <typename T>
__global__ void __launch_bounds__(kT) adj_generic_kernel(const T* __restrict__ K, sc_strides st, int Hkv, int n, int nb, int d,
                                                         float tau, const float* __restrict__ norms, uint32_t* __restrict__ bits) {
    __shared__ float As[kT][33], Bs[kT][33];
    const int I = blockIdx.x, j_begin = blockIdx.y * kJChunk, bh = blockIdx.z;
    if (j_begin > I) return;
    const int nt = min(kJChunk, I + 1 - j_begin);
    const int r = threadIdx.x, i = I * kT + r;
    const T* Kh = K + (bh / Hkv) * st.b + (bh % Hkv) * st.h;
    const float ni = i < n ? norms[(size_t)bh * n + i] : 0.f;
    const bool neg = tau < 0.f;
    uint32_t* row = bits + (size_t)bh * bits_words(nb) + tile_row_base(I) + (size_t)r * 4 * (I + 1);
    for (int t = 0; t < nt; ++t) {
        const int J = j_begin + t, jr = J * kT + r;
        float acc[kT];
#pragma unroll
        for (int j = 0; j < kT; ++j) acc[j] = 0.f;
        for (int c0 = 0; c0 < d; c0 += 32) {
            __syncthreads();
            for (int c = 0; c < 32; ++c) {
                As[r][c] = (i < n && c0 + c < d) ? Elem<T>::load(Kh + (long long)i * st.n + c0 + c) : 0.f;
                Bs[r][c] = (jr < n && c0 + c < d) ? Elem<T>::load(Kh + (long long)jr * st.n + c0 + c) : 0.f;
            }
            __syncthreads();
#pragma unroll 4
            for (int j = 0; j < kT; ++j) {
                float a = acc[j];
#pragma unroll
                for (int c = 0; c < 32; ++c) a = fmaf(As[r][c], Bs[j][c], a);
                acc[j] = a;
            }
        }
        uint32_t words[4] = {0u, 0u, 0u, 0u};
#pragma unroll
        for (int j = 0; j < kT; ++j) {
            const int jj = J * kT + j;
            const float nj = jj < n ? norms[(size_t)bh * n + jj] : 0.f;
            const float thr = ni * (tau * nj);
            bool hit = acc[j] > thr;
            if (neg) hit = hit || (thr == 0.f);
            if (hit && jj < i) words[j >> 5] |= 1u << (j & 31);
        }
        if (i < n) *reinterpret_cast<uint4*>(row + 4 * J) = make_uint4(words[0], words[1], words[2], words[3]);
    }
}

// Search state per call: ctl[r] = tokens still undecided when round r starts (ctl[0] = everything).
// Words of a head's token masks (seed, member, rank base): one bit per token, the stride rounded up to whole
// 16-byte groups so that a head's masks can be read four words at a time.
__host__ __device__ inline int mask_words(int n) { return (((n + 31) >> 5) + 3) & ~3; }

struct Masks {
    uint32_t* seed;      // [B*Hkv][nw]
    uint32_t* member;    // [B*Hkv][nw]
    int32_t* ctl;        // [kRounds + 2]
};

__global__ void init_kernel(Masks m, size_t words, long long tokens) {
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < words; i += (size_t)gridDim.x * blockDim.x) {
        m.seed[i] = 0u;
        m.member[i] = 0u;
    }
    if (blockIdx.x == 0 && threadIdx.x <= kRounds + 1) m.ctl[threadIdx.x] = threadIdx.x == 0 ? (tokens > 0x7fffffff ? 0x7fffffff : (int)tokens) : 0;
}

// One warp looks at one undecided token's earlier neighbours.  Returns 1 = seed, 2 = member, 0 = still open.
// The row's words come sixteen bytes per lane, two such reads in flight (a row of a 32K-token sequence is 4 KB: with
// one word per lane and a vote per 128 bytes the warp spent its time waiting for loads).  `words` is rounded up to
// the four-word groups the row is stored in; bits past the token's own position are zero there.
__device__ __forceinline__ int decide_row(const uint32_t* __restrict__ row, int words, const uint32_t* seed,
                                          const uint32_t* member, int lane) {
    const int groups = (words + 3) >> 2;
    const uint4* row4 = reinterpret_cast<const uint4*>(row);
    const uint4* seed4 = reinterpret_cast<const uint4*>(seed);
    const uint4* member4 = reinterpret_cast<const uint4*>(member);
    bool has_seed = false, has_open = false;
    for (int g0 = 0; g0 < groups; g0 += 64) {
        const int ga = g0 + lane, gb = g0 + 32 + lane;
        uint4 xa = make_uint4(0u, 0u, 0u, 0u), xb = xa;
        if (ga < groups) xa = __ldg(row4 + ga);
        if (gb < groups) xb = __ldg(row4 + gb);
        if (xa.x | xa.y | xa.z | xa.w) {
            const uint4 sd = __ldcg(seed4 + ga), mb = __ldcg(member4 + ga);   // through L2: other blocks add bits meanwhile
            has_seed |= ((xa.x & sd.x) | (xa.y & sd.y) | (xa.z & sd.z) | (xa.w & sd.w)) != 0u;
            has_open |= ((xa.x & ~(sd.x | mb.x)) | (xa.y & ~(sd.y | mb.y)) | (xa.z & ~(sd.z | mb.z)) | (xa.w & ~(sd.w | mb.w))) != 0u;
        }
        if (xb.x | xb.y | xb.z | xb.w) {
            const uint4 sd = __ldcg(seed4 + gb), mb = __ldcg(member4 + gb);
            has_seed |= ((xb.x & sd.x) | (xb.y & sd.y) | (xb.z & sd.z) | (xb.w & sd.w)) != 0u;
            has_open |= ((xb.x & ~(sd.x | mb.x)) | (xb.y & ~(sd.y | mb.y)) | (xb.z & ~(sd.z | mb.z)) | (xb.w & ~(sd.w | mb.w))) != 0u;
        }
        if (__any_sync(kFull, has_seed)) return 2;   // an earlier neighbour is a seed: final
    }
    return __any_sync(kFull, has_open) ? 0 : 1;      // every earlier neighbour is a member (or there is none): a seed
}

__global__ void __launch_bounds__(256) round_kernel(const uint32_t* __restrict__ bits, int n, int nb, int heads, Masks m, int round) {
    if (m.ctl[round] == 0) return;   // nothing left: uniform over the grid
    const int lane = threadIdx.x & 31;
    const int nw = mask_words(n);
    const long long rows = (long long)heads * n;
    int open = 0;
    for (long long rid = (long long)blockIdx.x * 8 + (threadIdx.x >> 5); rid < rows; rid += (long long)gridDim.x * 8) {
        const int bh = (int)(rid / n), i = (int)(rid - (long long)bh * n);
        uint32_t* seed = m.seed + (size_t)bh * nw;
        uint32_t* member = m.member + (size_t)bh * nw;
        const uint32_t bit = 1u << (i & 31);
        if ((((volatile uint32_t*)seed)[i >> 5] | ((volatile uint32_t*)member)[i >> 5]) & bit) continue;
        const int I = i / kT;
        const uint32_t* row = bits + (size_t)bh * bits_words(nb) + tile_row_base(I) + (size_t)(i - I * kT) * 4 * (I + 1);
        const int verdict = decide_row(row, (i + 31) >> 5, seed, member, lane);
        if (lane == 0) {
            if (verdict == 1) atomicOr(seed + (i >> 5), bit);
            else if (verdict == 2) atomicOr(member + (i >> 5), bit);
            else ++open;
        }
    }
    if (lane == 0 && open) atomicAdd(&m.ctl[round + 1], open);
}

// Whatever the enqueued rounds left open (long dependence chains): one block per head keeps going.  Each
// sweep decides at least the head's lowest open token, so n sweeps always suffice.
__global__ void __launch_bounds__(1024) finish_kernel(const uint32_t* __restrict__ bits, int n, int nb, Masks m) {
    if (m.ctl[kRounds] == 0) return;
    __shared__ int open_s;
    const int bh = blockIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int nw = mask_words(n);
    uint32_t* seed = m.seed + (size_t)bh * nw;
    uint32_t* member = m.member + (size_t)bh * nw;
    for (int sweep = 0; sweep <= n; ++sweep) {
        if (threadIdx.x == 0) open_s = 0;
        __syncthreads();
        int open = 0;
        for (int i = warp; i < n; i += 32) {
            const uint32_t bit = 1u << (i & 31);
            if ((((volatile uint32_t*)seed)[i >> 5] | ((volatile uint32_t*)member)[i >> 5]) & bit) continue;
            const int I = i / kT;
            const uint32_t* row = bits + (size_t)bh * bits_words(nb) + tile_row_base(I) + (size_t)(i - I * kT) * 4 * (I + 1);
            const int verdict = decide_row(row, (i + 31) >> 5, seed, member, lane);
            if (lane == 0) {
                if (verdict == 1) atomicOr(seed + (i >> 5), bit);
                else if (verdict == 2) atomicOr(member + (i >> 5), bit);
                else ++open;
            }
        }
        if (lane == 0 && open) atomicAdd(&open_s, open);
        __syncthreads();
        if (open_s == 0) break;
        __syncthreads();
    }
}

// Step 4a: ranks of the seeds (exclusive prefix sum of the seed bits per head) and core_len.
__global__ void __launch_bounds__(1024) rank_kernel(const uint32_t* __restrict__ seed, int n, int32_t* __restrict__ rank_base,
                                                    int32_t* __restrict__ core_len, int cap, int32_t* status) {
    __shared__ int wsum[32];
    const int bh = blockIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int nw = mask_words(n);
    int carry = 0;
    for (int base = 0; base < nw; base += 1024) {
        const int w = base + threadIdx.x;
        const int v = w < nw ? __popc(seed[(size_t)bh * nw + w]) : 0;
        const int incl = warp_scan_add(v, lane);
        if (lane == 31) wsum[warp] = incl;
        __syncthreads();
        int pre = 0, tot = 0;
        for (int k = 0; k < 32; ++k) { if (k < warp) pre += wsum[k]; tot += wsum[k]; }
        __syncthreads();
        if (w < nw) rank_base[(size_t)bh * nw + w] = carry + pre + incl - v;
        carry += tot;
    }
    if (threadIdx.x == 0) {
        core_len[bh] = carry;
        if (carry > cap) set_status(status, SC_ERR_CAPACITY);
    }
}

// Step 4b: every token's seed: itself, or the lowest earlier neighbour that is a seed.
__global__ void __launch_bounds__(256) assign_kernel(const uint32_t* __restrict__ bits, int n, int nb, int heads,
                                                     const uint32_t* __restrict__ seed, int32_t* __restrict__ assign) {
    const int lane = threadIdx.x & 31;
    const int nw = mask_words(n);
    const long long rows = (long long)heads * n;
    for (long long rid = (long long)blockIdx.x * 8 + (threadIdx.x >> 5); rid < rows; rid += (long long)gridDim.x * 8) {
        const int bh = (int)(rid / n), i = (int)(rid - (long long)bh * n);
        const uint32_t* sd = seed + (size_t)bh * nw;
        if ((sd[i >> 5] >> (i & 31)) & 1u) {
            if (lane == 0) assign[rid] = i;
            continue;
        }
        const int I = i / kT;
        const uint32_t* row = bits + (size_t)bh * bits_words(nb) + tile_row_base(I) + (size_t)(i - I * kT) * 4 * (I + 1);
        const int groups = (((i + 31) >> 5) + 3) >> 2;   // the row in its four-word groups, sixteen bytes per lane
        const uint4* row4 = reinterpret_cast<const uint4*>(row);
        const uint4* sd4 = reinterpret_cast<const uint4*>(sd);
        int found = -1;
        for (int g0 = 0; g0 < groups && found < 0; g0 += 32) {
            const int g = g0 + lane;
            uint4 x = make_uint4(0u, 0u, 0u, 0u);
            if (g < groups) {
                const uint4 rw = __ldg(row4 + g), sw = __ldg(sd4 + g);
                x = make_uint4(rw.x & sw.x, rw.y & sw.y, rw.z & sw.z, rw.w & sw.w);
            }
            const uint32_t vote = __ballot_sync(kFull, (x.x | x.y | x.z | x.w) != 0u);
            if (vote) {
                const int src = __ffs(vote) - 1;
                const uint32_t x0 = __shfl_sync(kFull, x.x, src), x1 = __shfl_sync(kFull, x.y, src);
                const uint32_t x2 = __shfl_sync(kFull, x.z, src), x3 = __shfl_sync(kFull, x.w, src);
                const int sub = x0 ? 0 : (x1 ? 1 : (x2 ? 2 : 3));
                const uint32_t xs = x0 ? x0 : (x1 ? x1 : (x2 ? x2 : x3));
                found = ((g0 + src) * 4 + sub) * 32 + __ffs(xs) - 1;
            }
        }
        if (lane == 0) assign[rid] = found;   // a member always has one
    }
}

// Step 5a: cluster index of a token = rank of its seed among the head's seeds.
__device__ __forceinline__ int cluster_of(const uint32_t* __restrict__ seed, const int32_t* __restrict__ rank_base, int seed_pos) {
    const uint32_t sw = seed[seed_pos >> 5];
    return rank_base[seed_pos >> 5] + __popc(sw & ((1u << (seed_pos & 31)) - 1u));
}

// Step 5b: cluster sizes (phase 0), then every token into its cluster's slice of the member list (phase 1).
// The order inside a slice is whatever the atomics gave; the pooling kernel puts it right.
__global__ void __launch_bounds__(256) members_kernel(int n, int heads, const uint32_t* __restrict__ seed,
                                                      const int32_t* __restrict__ rank_base, const int32_t* __restrict__ assign,
                                                      int32_t* __restrict__ csize, const int32_t* __restrict__ coff,
                                                      int32_t* __restrict__ cursor, int32_t* __restrict__ members, int phase) {
    const int nw = mask_words(n);
    const long long rows = (long long)heads * n;
    for (long long rid = (long long)blockIdx.x * blockDim.x + threadIdx.x; rid < rows; rid += (long long)gridDim.x * blockDim.x) {
        const int bh = (int)(rid / n), j = (int)(rid - (long long)bh * n);
        const int c = cluster_of(seed + (size_t)bh * nw, rank_base + (size_t)bh * nw, assign[rid]);
        if (phase == 0) atomicAdd(&csize[(size_t)bh * n + c], 1);
        else members[(size_t)bh * n + coff[(size_t)bh * n + c] + atomicAdd(&cursor[(size_t)bh * n + c], 1)] = j;
    }
}

// Step 5c: exclusive prefix sum of the cluster sizes per head.
__global__ void __launch_bounds__(1024) offsets_kernel(int n, const int32_t* __restrict__ core_len, const int32_t* __restrict__ csize,
                                                       int32_t* __restrict__ coff) {
    __shared__ int wsum[32];
    const int bh = blockIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int S = min(core_len[bh], n);
    int carry = 0;
    for (int base = 0; base < S; base += 1024) {
        const int c = base + threadIdx.x;
        const int v = c < S ? csize[(size_t)bh * n + c] : 0;
        const int incl = warp_scan_add(v, lane);
        if (lane == 31) wsum[warp] = incl;
        __syncthreads();
        int pre = 0, tot = 0;
        for (int k = 0; k < 32; ++k) { if (k < warp) pre += wsum[k]; tot += wsum[k]; }
        __syncthreads();
        if (c < S) coff[(size_t)bh * n + c] = carry + pre + incl - v;
        carry += tot;
    }
}

// Step 5d (Eq. 3): one warp per cluster pools its members in token order (fp32 sums, one divide, one rounding).
// Up to 32 members are ordered in registers; up to kMidCluster by repeatedly taking the next larger position;
// beyond that the warp walks the head's assignment array, which is already in token order.
constexpr int kMidCluster = 1024;
template <typename T>
__device__ __forceinline__ void add_row(const T* __restrict__ Kh, const T* __restrict__ Vh, long long sn, int jj, int d, int lane,
                                        float (&sk)[8], float (&sv)[8]) {
    const T* kr = Kh + (long long)jj * sn;
    const T* vr = Vh + (long long)jj * sn;
#pragma unroll
    for (int u = 0; u < 8; ++u) {
        const int c = lane + 32 * u;
        if (c < d) { sk[u] += Elem<T>::load(kr + c); sv[u] += Elem<T>::load(vr + c); }
    }
}

template <typename T>
__global__ void __launch_bounds__(256) merge_kernel(const T* __restrict__ K, const T* __restrict__ V, sc_strides st, int Hkv, int n,
                                                    int d, int heads, const int32_t* __restrict__ core_len,
                                                    const int32_t* __restrict__ csize, const int32_t* __restrict__ coff,
                                                    const int32_t* __restrict__ members, const int32_t* __restrict__ assign,
                                                    T* __restrict__ core_k, T* __restrict__ core_v, int32_t* __restrict__ count, int cap) {
    const int lane = threadIdx.x & 31;
    const long long slots = (long long)heads * n;
    for (long long sid = (long long)blockIdx.x * 8 + (threadIdx.x >> 5); sid < slots; sid += (long long)gridDim.x * 8) {
        const int bh = (int)(sid / n), c = (int)(sid - (long long)bh * n);
        if (c >= min(core_len[bh], cap)) continue;
        const T* Kh = K + (bh / Hkv) * st.b + (bh % Hkv) * st.h;
        const T* Vh = V + (bh / Hkv) * st.b + (bh % Hkv) * st.h;
        const int cnt = csize[(size_t)bh * n + c];
        const int32_t* mem = members + (size_t)bh * n + coff[(size_t)bh * n + c];
        float sk[8], sv[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) sk[u] = sv[u] = 0.f;
        if (cnt <= 32) {
            const int mine = lane < cnt ? mem[lane] : 0x7fffffff;
            int pos = 0;
            for (int k = 0; k < cnt; ++k) pos += __shfl_sync(kFull, mine, k) < mine;
            for (int t = 0; t < cnt; ++t) {
                const int src = __ffs(__ballot_sync(kFull, lane < cnt && pos == t)) - 1;
                add_row<T>(Kh, Vh, st.n, __shfl_sync(kFull, mine, src), d, lane, sk, sv);
            }
        } else if (cnt <= kMidCluster) {
            int last = -1;
            for (int t = 0; t < cnt; ++t) {
                int best = 0x7fffffff;
                for (int k = lane; k < cnt; k += 32) { const int v = mem[k]; if (v > last && v < best) best = v; }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) best = min(best, __shfl_xor_sync(kFull, best, o));
                add_row<T>(Kh, Vh, st.n, best, d, lane, sk, sv);
                last = best;
            }
        } else {
            const int32_t* as = assign + (size_t)bh * n;
            int seed_pos = 0x7fffffff;   // the cluster's seed is its smallest member
            for (int k = lane; k < cnt; k += 32) seed_pos = min(seed_pos, mem[k]);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) seed_pos = min(seed_pos, __shfl_xor_sync(kFull, seed_pos, o));
            for (int j0 = seed_pos & ~31; j0 < n; j0 += 32) {
                const int j = j0 + lane;
                uint32_t hit = __ballot_sync(kFull, j < n && as[j] == seed_pos);
                while (hit) {
                    add_row<T>(Kh, Vh, st.n, j0 + __ffs(hit) - 1, d, lane, sk, sv);
                    hit &= hit - 1;
                }
            }
        }
        const size_t o = ((size_t)bh * cap + c) * d;
        const float fc = (float)cnt;
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int col = lane + 32 * u;
            if (col < d) {
                Elem<T>::store(core_k + o + col, sk[u] / fc);
                Elem<T>::store(core_v + o + col, sv[u] / fc);
            }
        }
        if (lane == 0) count[(size_t)bh * cap + c] = cnt;
    }
}

struct Layout {   // workspace: every part 256-byte aligned
    size_t norms, bits, seed, member, rank, assign, csize, coff, members, ctl, total;
};
inline Layout layout_for(int B, int Hkv, int n) {
    const size_t heads = (size_t)B * Hkv, nb = (n + kT - 1) / kT, nw = mask_words(n);
    auto up = [](size_t x) { return (x + 255) / 256 * 256; };
    Layout L;
    size_t off = 0;
    L.norms = off; off += up(4 * heads * n);
    L.bits = off; off += up(4 * heads * bits_words(nb));
    L.seed = off; off += up(4 * heads * nw);
    L.member = off; off += up(4 * heads * nw);
    L.rank = off; off += up(4 * heads * nw);
    L.assign = off; off += up(4 * heads * n);
    L.csize = off; off += 2 * up(4 * heads * n);      // cluster sizes, then the fill cursors (cleared together)
    L.coff = off; off += up(4 * heads * n);
    L.members = off; off += up(4 * heads * n);
    L.ctl = off; off += 256;
    L.total = off;
    return L;
}

}  // namespace gl

size_t compress_global_ws_bytes(int32_t B, int32_t Hkv, int32_t n) { return gl::layout_for(B, Hkv, n).total; }

template <typename T>
static cudaError_t run_global(const GlobalArgs& a, cudaStream_t st) {
    using namespace gl;
    const Layout L = layout_for(a.B, a.Hkv, a.n);
    char* ws = (char*)a.ws;
    float* norms = (float*)(ws + L.norms);
    uint32_t* bits = (uint32_t*)(ws + L.bits);
    Masks m{(uint32_t*)(ws + L.seed), (uint32_t*)(ws + L.member), (int32_t*)(ws + L.ctl)};
    int32_t* rank_base = (int32_t*)(ws + L.rank);
    int32_t* assign = a.assign ? a.assign : (int32_t*)(ws + L.assign);
    const int heads = a.B * a.Hkv, nb = (a.n + kT - 1) / kT, nw = mask_words(a.n);
    const long long rows = (long long)heads * a.n;
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);

    norms_kernel<T><<<div_up(rows, 8), 256, 0, st>>>((const T*)a.K, a.st, a.Hkv, a.n, a.d, rows, norms);
    init_kernel<<<sms, 256, 0, st>>>(m, (size_t)heads * nw, rows);
    int launched = 2;

    const dim3 grid(nb, div_up(nb, kJChunk), heads);
    bool umma_done = false;
    if (a.dt == SC_BF16 && a.d == 128 && !(a.flags & SC_FLAG_GENERIC) && heads <= 65535 && nb <= 65535) {
        static bool attr_set[64] = {false};
        if (!attr_set[dev & 63]) {
            cudaFuncSetAttribute(adj_umma_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
            cudaFuncSetAttribute(adj_umma_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
            attr_set[dev & 63] = true;
        }
        AdjParams p;
        p.norms = norms; p.bits = bits; p.n = a.n; p.nb = nb; p.Hkv = a.Hkv; p.tau = a.tau; p.status = a.status;
        if (make_map_bf16_rows(&p.map, a.K, a.st.b, a.st.h, a.st.n, a.B, a.Hkv, a.n, kT)) {
            if (a.tau < 0.f) adj_umma_kernel<true><<<grid, kThreads, kSmemBytes, st>>>(p);
            else adj_umma_kernel<false><<<grid, kThreads, kSmemBytes, st>>>(p);
            umma_done = true;
        }
    }
    if (!umma_done)
        adj_generic_kernel<T><<<grid, kT, 0, st>>>((const T*)a.K, a.st, a.Hkv, a.n, nb, a.d, a.tau, norms, bits);
    ++launched;

    const int round_grid = (int)(rows / 8 < (long long)sms * 16 ? (rows + 7) / 8 : (long long)sms * 16);
    for (int r = 0; r < kRounds; ++r) round_kernel<<<round_grid, 256, 0, st>>>(bits, a.n, nb, heads, m, r);
    finish_kernel<<<heads, 1024, 0, st>>>(bits, a.n, nb, m);
    rank_kernel<<<heads, 1024, 0, st>>>(m.seed, a.n, rank_base, a.core_len, a.cap, a.status);
    assign_kernel<<<round_grid, 256, 0, st>>>(bits, a.n, nb, heads, m.seed, assign);
    auto up = [](size_t x) { return (x + 255) / 256 * 256; };
    int32_t* csize = (int32_t*)(ws + L.csize);
    int32_t* cursor = (int32_t*)(ws + L.csize + up(4 * (size_t)heads * a.n));
    int32_t* coff = (int32_t*)(ws + L.coff);
    int32_t* members = (int32_t*)(ws + L.members);
    cudaMemsetAsync(csize, 0, 2 * up(4 * (size_t)heads * a.n), st);
    const int tok_grid = (int)(rows / 256 < (long long)sms * 8 ? (rows + 255) / 256 : (long long)sms * 8);
    members_kernel<<<tok_grid, 256, 0, st>>>(a.n, heads, m.seed, rank_base, assign, csize, coff, cursor, members, 0);
    offsets_kernel<<<heads, 1024, 0, st>>>(a.n, a.core_len, csize, coff);
    members_kernel<<<tok_grid, 256, 0, st>>>(a.n, heads, m.seed, rank_base, assign, csize, coff, cursor, members, 1);
    merge_kernel<T><<<round_grid, 256, 0, st>>>((const T*)a.K, (const T*)a.V, a.st, a.Hkv, a.n, a.d, heads, a.core_len, csize, coff,
                                                members, assign, (T*)a.core_k, (T*)a.core_v, a.count, a.cap);
    note_launches(launched + kRounds + 7);
    return cudaGetLastError();
}

cudaError_t launch_compress_global(const GlobalArgs& a, cudaStream_t st) {
    return a.dt == SC_BF16 ? run_global<__nv_bfloat16>(a, st) : run_global<float>(a, st);
}

}  // namespace sc
