// Multi-query Proportional Attention (Sec. 2.4, Eq. 4 as printed, with a block of m queries per head):
//     O = softmax(Q K_c^T * scale + ln s) V_c      Q: [m, d] per query head, K_c/V_c: the head's cores
// for chunked prefill or speculative decoding over a compressed cache.  Unlike the one-query decode
// step this is a dense contraction: the G query heads that share a KV head times the m queries give
// G*m rows against the same cores, so it runs on the tcgen05 tensor cores (bf16, d = 128):
//   one CTA = 128 query rows of one (sequence, KV head), walking the head's cores 128 at a time;
//   warp 0     TMA: the query tile once, then K and V tiles into a three-stage ring (128-byte swizzle);
//   warp 1     issues the MMAs: S = Q K^T into one of two score buffers in tensor memory (two tiles ahead
//              of the weighted sum), then O += P V with P read from tensor memory and V as an MN-major
//              operand straight from its [keys x dims] tile;
//   warps 2-9  softmax, two threads per query row (= tensor-memory lane; each owns half of a tile's keys and
//              half of the accumulator's columns, the row maximum is exchanged through shared memory):
//              x = S * scale*log2(e) + log2(count), masks (head length, optional causal tail), running
//              maximum raised lazily (the accumulator row is rescaled in tensor memory only then; the tile's
//              maximum is taken as a bound: largest raw product * scale + largest log2(count) of the tile),
//              P = 2^(x - m) as a bf16 pair (leading part + remainder) written back over the scores it
//              came from: the 32 fp32 columns of a chunk of scores become 16 columns of packed leading
//              parts and 16 of remainders, so P is double-buffered like S and never touches shared
//              memory; finally O / l -> bf16 -> global.
// When the launch has too few CTAs to fill the GPU (few query rows: speculative decoding, short chunks), the keys
// of a head are split over the CTAs of a thread-block cluster: each walks its share of the key tiles, leaves its
// unnormalised (m, l, O) in its own shared memory, and after a cluster barrier every CTA folds a slice of the
// query rows out of all members' shared memory (distributed shared memory) and writes that slice of the output.
// Every wait is bounded; a wait that gives up is reported through the status word.
// A CUDA-core kernel (one warp per query) serves other dtypes and head sizes.
#include <cooperative_groups.h>

#include "common.cuh"
#include "umma.cuh"

namespace sc {

namespace pf {

using namespace umma;
namespace cg = cooperative_groups;

constexpr int kT = 128;                       // query rows per CTA, keys per tile
constexpr int kHalf = kT * 128;               // 16384 bytes: one 64-column half of a [128 x 128] bf16 tile
constexpr int kTile = 2 * kHalf;              // 32768
constexpr int kThreads = 320;                 // warp 0: TMA, warp 1: MMA + tensor memory, warps 2-9: softmax
constexpr int kTmemCols = 512;                // S0 | S1 | O (128 columns each; P overwrites S in place), rounded up to a power of two
constexpr int kColS = 0, kColO = 256;
constexpr int kStages = 3;                    // K/V ring
constexpr int kSmQ = 0, kSmK = kTile, kSmV = (1 + kStages) * kTile, kSmLc = (1 + 2 * kStages) * kTile, kSmMx = kSmLc + 2 * kT * 4,
              kSmBar = kSmMx + 2 * kT * 4;
constexpr int kSmemBytes = kSmBar + 256;
constexpr int kMaxSplit = 8;                  // portable cluster size
constexpr float kMaxSlack = 8.f;              // log2 units a score may exceed the running maximum before it is raised
static_assert(kSmemBytes <= 232448, "shared memory of one CTA");

struct Params {
    CUtensorMap map_q, map_k, map_v;          // rows x 128 bf16, boxes of 128 rows x 64 columns
    const int32_t* count; const int32_t* core_len;
    __nv_bfloat16* out;
    int Hq, Hkv, m, cap, causal, n_split;   // n_split: CTAs (= cluster size) that share the keys of one query tile
    float scale_log2;
    int32_t* status;
};

__device__ __forceinline__ float ex2(float x) { float y; asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x)); return y; }
__device__ __forceinline__ float lg2(float x) { float y; asm("lg2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x)); return y; }
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};\n"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
          "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
          "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};\n"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]: A's rows are tensor-memory lanes, two 16-bit elements of the contraction
// axis per 32-bit column; one thread issues.
__device__ __forceinline__ void mma_bf16_ts(uint32_t tmem_d, uint32_t tmem_a, uint64_t bdesc, uint32_t idesc, bool accumulate) {
    asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n}\n"
                 ::"r"(tmem_d), "r"(tmem_a), "l"(bdesc), "r"(idesc), "r"((uint32_t)accumulate) : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;\n" ::: "memory"); }
__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}
// r0 = w0 - low bf16 of ph, r1 = w1 - high bf16 of ph, with the mixed-precision fma (the bf16 operands are taken
// as they are: (-1) * h + w, one rounding -- what unpacking and subtracting gives, in half the instructions).
__device__ __forceinline__ void remainders(uint32_t ph, float w0, float w1, float& r0, float& r1) {
    asm("{\n.reg .b16 lo, hi, m1;\nmov.b32 {lo, hi}, %2;\nmov.b16 m1, 0xBF80;\n"
        "fma.rn.f32.bf16 %0, lo, m1, %3;\nfma.rn.f32.bf16 %1, hi, m1, %4;\n}\n"
        : "=f"(r0), "=f"(r1) : "r"(ph), "f"(w0), "f"(w1));
}
__device__ __forceinline__ float bf_lo(uint32_t v) { return __uint_as_float(v << 16); }
__device__ __forceinline__ float bf_hi(uint32_t v) { return __uint_as_float(v & 0xffff0000u); }

__global__ void __launch_bounds__(kThreads, 1) prefill_umma_kernel(const __grid_constant__ Params p) {
    extern __shared__ __align__(1024) unsigned char smem[];   // the swizzle pattern repeats every 1024 bytes
    const int n_split = p.n_split, split = blockIdx.x % n_split;   // the CTAs of a cluster are consecutive in x
    const int qt = blockIdx.x / n_split, h = blockIdx.y, b = blockIdx.z;
    const int G = p.Hq / p.Hkv, bh = b * p.Hkv + h;
    const int rows_total = G * p.m;                           // query rows of this (sequence, KV head)
    const int len = max(min(p.core_len[bh], p.cap), 0);
    const int nt_all = (len + kT - 1) / kT;                   // key tiles of the head
    const int per_split = (nt_all + n_split - 1) / n_split;
    const int t_lo = min(split * per_split, nt_all);          // this CTA's tiles: [t_lo, t_lo + nt)
    const int nt = min(t_lo + per_split, nt_all) - t_lo;
    const long long q_row0 = ((long long)b * p.Hq + (long long)h * G) * p.m + (long long)qt * kT;
    const uint32_t sbase = smem_u32(smem);
    if ((sbase & 1023u) != 0u) {   // the swizzled addressing assumes this; uniform over the block
        if (threadIdx.x == 0) set_status(p.status, SC_ERR_CUDA);
        return;
    }
    float* lc_s = reinterpret_cast<float*>(smem + kSmLc);     // [2][128] log2(count) of the tile's keys
    float* mx_s = reinterpret_cast<float*>(smem + kSmMx);     // [2][128] each half's row maximum (at the end the row sums)
    int* lcm_s = reinterpret_cast<int*>(smem + kSmBar + 128);  // [2][4] largest log2(count) of a tile, per writing warp (float bits)
    const uint32_t bar0 = sbase + kSmBar;
    const uint32_t q_full = bar0, kv_full0 = bar0 + 8, kv_empty0 = bar0 + 32, s_full0 = bar0 + 56, p_full0 = bar0 + 72,
                   pv_done0 = bar0 + 88;
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + kSmBar + 104);
    volatile int* sh_fail = reinterpret_cast<volatile int*>(smem + kSmBar + 108);
    volatile int* sh_fail_sm = reinterpret_cast<volatile int*>(smem + kSmBar + 112);   // set by the softmax warps only
    volatile int* sh_issued = reinterpret_cast<volatile int*>(smem + kSmBar + 116);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        mbar_init(q_full, 1);
        for (int s = 0; s < kStages; ++s) {
            mbar_init(kv_full0 + 8 * s, 1);
            mbar_init(kv_empty0 + 8 * s, 1);
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(s_full0 + 8 * s, 1);
            mbar_init(p_full0 + 8 * s, 8);
            mbar_init(pv_done0 + 8 * s, 1);
        }
        mbar_fence_init();
        *sh_fail = 0; *sh_fail_sm = 0; *sh_issued = 0;
    }
    if (warp == 1) tmem_alloc(sbase + kSmBar + 104, kTmemCols);
    fence_before_sync();
    __syncthreads();
    fence_after_sync();
    const uint32_t tmem = *tmem_slot;

    if (warp == 0) {
        if (lane == 0 && nt > 0) {   // ---- TMA producer ----
            mbar_expect_tx(q_full, kTile);
            tma_load_4d(sbase + kSmQ, &p.map_q, 0, (int)q_row0, 0, 0, q_full);
            tma_load_4d(sbase + kSmQ + kHalf, &p.map_q, 64, (int)q_row0, 0, 0, q_full);
            const int row_base = bh * p.cap + t_lo * kT;
            for (int t = 0; t < nt; ++t) {
                const int s = t % kStages;
                if (t >= kStages && !mbar_wait(kv_empty0 + 8 * s, ((t / kStages) - 1) & 1)) { *sh_fail = 1; break; }
                mbar_expect_tx(kv_full0 + 8 * s, 2 * kTile);
                const uint32_t dk = sbase + kSmK + s * kTile, dv = sbase + kSmV + s * kTile;
                tma_load_4d(dk, &p.map_k, 0, row_base + t * kT, 0, 0, kv_full0 + 8 * s);
                tma_load_4d(dk + kHalf, &p.map_k, 64, row_base + t * kT, 0, 0, kv_full0 + 8 * s);
                tma_load_4d(dv, &p.map_v, 0, row_base + t * kT, 0, 0, kv_full0 + 8 * s);
                tma_load_4d(dv + kHalf, &p.map_v, 64, row_base + t * kT, 0, 0, kv_full0 + 8 * s);
                *sh_issued = t + 1;
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && nt > 0) {   // ---- MMA issuer ----
            constexpr uint32_t idesc_qk = instr_desc_bf16(kT, kT, false, false);   // Q and K both K-major
            constexpr uint32_t idesc_pv = instr_desc_bf16(kT, kT, false, true);    // P K-major (tensor memory), V MN-major
            const uint32_t aq = sbase + kSmQ;
            auto issue_qk = [&](int t) {   // S[t & 1] = Q K_t^T
                const uint32_t bk = sbase + kSmK + (t % kStages) * kTile;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    const uint32_t off = (ks >> 2) * kHalf + (ks & 3) * 32;
                    mma_bf16_ss(tmem + kColS + (t & 1) * kT, smem_desc_sw128(aq + off, 16, 1024), smem_desc_sw128(bk + off, 16, 1024),
                                idesc_qk, ks > 0);
                }
                mma_commit(s_full0 + 8 * (t & 1));
            };
            bool ok = mbar_wait(q_full, 0) && mbar_wait(kv_full0, 0);
            if (ok) { fence_after_sync(); issue_qk(0); }
            if (ok && nt > 1) {
                ok = mbar_wait(kv_full0 + 8, 0);
                if (ok) { fence_after_sync(); issue_qk(1); }
            }
            for (int t = 0; t < nt && ok; ++t) {
                const int sb = t & 1;
                ok = mbar_wait(p_full0 + 8 * sb, (t >> 1) & 1);   // the weights of tile t are in tensor memory
                if (!ok) break;
                fence_after_sync();
                const uint32_t bv = sbase + kSmV + (t % kStages) * kTile;
                const uint32_t pcol = tmem + kColS + sb * kT;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {   // sixteen keys per instruction: eight packed columns of P
                    const uint64_t vdesc = smem_desc_sw128(bv + ks * 16 * 128, kHalf, 1024);   // V: MN-major, 16 key rows down
                    const uint32_t pa = pcol + (ks >> 1) * 32 + (ks & 1) * 8;                  // leading parts; remainders 16 columns on
                    mma_bf16_ts(tmem + kColO, pa, vdesc, idesc_pv, t > 0 || ks > 0);
                    mma_bf16_ts(tmem + kColO, pa + 16, vdesc, idesc_pv, true);
                }
                mma_commit(kv_empty0 + 8 * (t % kStages));   // K and V of this stage are spent
                mma_commit(pv_done0 + 8 * sb);               // P of this buffer is spent, O holds tile t
                if (t + 2 < nt) {   // the scores two tiles ahead go where this tile's scores and weights were
                    ok = mbar_wait(kv_full0 + 8 * ((t + 2) % kStages), ((t + 2) / kStages) & 1) &&
                         mbar_wait(pv_done0 + 8 * sb, (t >> 1) & 1);
                    if (!ok) break;
                    fence_after_sync();
                    issue_qk(t + 2);
                }
            }
            if (!ok) *sh_fail = 1;
        }
    } else {
        // ---- softmax: two threads per query row (= tensor-memory lane), each owning 64 of a tile's 128 keys
        //      and 64 of the accumulator's 128 columns; warps 2-5 take the first halves, warps 6-9 the second ----
        const int q = warp & 3, r = q * 32 + lane, wg = (warp - 2) >> 2;
        const int row = qt * kT + r;                          // row among the G*m of this head group
        const bool row_ok = row < rows_total;
        const int qi = row % p.m;                             // which of the m queries
        const int vis = p.causal ? len - (p.m - 1 - qi) : len;   // keys this row sees: [0, vis)
        const uint32_t lane_addr = tmem + ((uint32_t)(q * 32) << 16);
        const int32_t* cnt = p.count ? p.count + (size_t)bh * p.cap : nullptr;
        float m_run = -INFINITY, l_run = 0.f;                 // l_run: this thread's keys only
        bool failed = false;
        for (int t = 0; t < nt; ++t) {
            const int s = t & 1, st = t % kStages, j0 = (t_lo + t) * kT, jw = j0 + wg * 64;   // jw: first key of this thread's half
            if (wg == 0) {
                const float lc = (cnt != nullptr && j0 + r < len) ? lg2((float)max(cnt[j0 + r], 1)) : 0.f;
                lc_s[s * kT + r] = lc;
                const int top = __reduce_max_sync(kFull, __float_as_int(lc));   // lc >= 0: the bits order like the values
                if (lane == 0) lcm_s[s * 4 + q] = top;
            }
            if (!mbar_wait(s_full0 + 8 * s, (t >> 1) & 1)) { *sh_fail = 1; *sh_fail_sm = 1; }
            fence_after_sync();
            asm volatile("bar.sync 1, 256;\n" ::: "memory");   // the eight softmax warps: log2(count) is in place
            if (*sh_fail_sm) { failed = true; break; }
            // Rows of the stage past the head's end hold whatever lies behind the cores (0 * NaN would poison
            // the second product): this row's threads clear its V row.  K rows need nothing, their scores are masked.
            if (j0 + r >= len) {
#pragma unroll
                for (int u = 0; u < 8; ++u)
                    *reinterpret_cast<uint4*>(smem + kSmV + st * kTile + wg * kHalf + r * 128 + u * 16) = make_uint4(0u, 0u, 0u, 0u);
            }
            // pass 1: a bound on the row's largest score in this tile (each thread its half, then the two are
            // exchanged): the largest raw product times the scale plus the tile's largest log2(count).  Any reference
            // at or above the true maximum serves the softmax; this one is at most log2 of the largest count above it,
            // and costs one instruction per score.  (A scale that is not positive takes the exact form.)
            float mx = -INFINITY;
            const bool all_seen = __all_sync(kFull, jw + 64 <= vis);   // no key of this half is masked for any row of the warp
            const bool exact = !(p.scale_log2 > 0.f);
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                uint32_t g[32];
                tmem_ld32(lane_addr + kColS + s * kT + wg * 64 + c * 32, g);
                tmem_ld_wait();
                if (exact) {
#pragma unroll
                    for (int k = 0; k < 32; ++k) {
                        const float x = fmaf(__uint_as_float(g[k]), p.scale_log2, lc_s[s * kT + wg * 64 + c * 32 + k]);
                        if (jw + c * 32 + k < vis) mx = fmaxf(mx, x);
                    }
                } else if (all_seen) {
#pragma unroll
                    for (int k = 0; k < 32; ++k) mx = fmaxf(mx, __uint_as_float(g[k]));
                } else {
#pragma unroll
                    for (int k = 0; k < 32; ++k)
                        if (jw + c * 32 + k < vis) mx = fmaxf(mx, __uint_as_float(g[k]));
                }
            }
            if (!exact && mx != -INFINITY) {
                const int top = max(max(lcm_s[s * 4], lcm_s[s * 4 + 1]), max(lcm_s[s * 4 + 2], lcm_s[s * 4 + 3]));
                mx = fmaf(mx, p.scale_log2, __int_as_float(top));
            }
            mx_s[wg * kT + r] = mx;
            asm volatile("bar.sync 2, 256;\n" ::: "memory");   // both halves' maxima are in place
            mx = fmaxf(mx, mx_s[(wg ^ 1) * kT + r]);
            const bool raise = mx > m_run + kMaxSlack;      // also the first finite score (m_run = -inf); same in both threads
            if (__any_sync(kFull, raise)) {
                const float f = raise ? ex2(m_run - mx) : 1.f;   // 0 when nothing had been seen
                // the accumulator may be touched only between two weighted sums: the previous one must be complete
                // (this tile's cannot start before this warp has handed in its weights)
                if (t > 0 && !mbar_wait(pv_done0 + 8 * ((t - 1) & 1), ((t - 1) >> 1) & 1)) { *sh_fail = 1; *sh_fail_sm = 1; }
                fence_after_sync();
                if (t > 0) {
#pragma unroll
                    for (int c = 0; c < 2; ++c) {
                        uint32_t o[32];
                        tmem_ld32(lane_addr + kColO + wg * 64 + c * 32, o);
                        tmem_ld_wait();
#pragma unroll
                        for (int k = 0; k < 32; ++k) o[k] = __float_as_uint(__uint_as_float(o[k]) * f);
                        tmem_st32(lane_addr + kColO + wg * 64 + c * 32, o);
                    }
                    tmem_st_wait();
                }
                l_run *= f;
                if (raise) m_run = mx;
            }
            // pass 2: weights, as bf16 pairs (leading part + remainder), back into the score buffer's columns
            const float mref = m_run == -INFINITY ? 0.f : m_run;
            // (the row sum takes the weights before the split: the pair carries sixteen bits of each, the difference
            // is below 2^-17 of the sum)
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                uint32_t g[32];
                tmem_ld32(lane_addr + kColS + s * kT + wg * 64 + c * 32, g);
                tmem_ld_wait();
                uint32_t hi[16], lo[16];
                if (all_seen) {   // no key of this half is masked for any row of the warp
#pragma unroll
                    for (int k = 0; k < 32; k += 2) {
                        const float x0 = fmaf(__uint_as_float(g[k]), p.scale_log2, lc_s[s * kT + wg * 64 + c * 32 + k]);
                        const float x1 = fmaf(__uint_as_float(g[k + 1]), p.scale_log2, lc_s[s * kT + wg * 64 + c * 32 + k + 1]);
                        const float w0 = ex2(x0 - mref), w1 = ex2(x1 - mref);
                        const uint32_t ph = pack2(w0, w1);
                        float r0, r1;
                        remainders(ph, w0, w1, r0, r1);
                        l_run += w0 + w1;
                        hi[k >> 1] = ph; lo[k >> 1] = pack2(r0, r1);
                    }
                } else {
#pragma unroll
                    for (int k = 0; k < 32; k += 2) {
                        const float x0 = fmaf(__uint_as_float(g[k]), p.scale_log2, lc_s[s * kT + wg * 64 + c * 32 + k]);
                        const float x1 = fmaf(__uint_as_float(g[k + 1]), p.scale_log2, lc_s[s * kT + wg * 64 + c * 32 + k + 1]);
                        const float w0 = (jw + c * 32 + k < vis) ? ex2(x0 - mref) : 0.f;
                        const float w1 = (jw + c * 32 + k + 1 < vis) ? ex2(x1 - mref) : 0.f;
                        const uint32_t ph = pack2(w0, w1);
                        float r0, r1;
                        remainders(ph, w0, w1, r0, r1);
                        l_run += w0 + w1;
                        hi[k >> 1] = ph; lo[k >> 1] = pack2(r0, r1);
                    }
                }
                // the 32 score columns just read become 16 columns of packed leading parts and 16 of remainders
                tmem_st16(lane_addr + kColS + s * kT + wg * 64 + c * 32, hi);
                tmem_st16(lane_addr + kColS + s * kT + wg * 64 + c * 32 + 16, lo);
            }
            tmem_st_wait();
            fence_before_sync();      // this thread's accesses to tensor memory
            fence_async_proxy();      // a cleared V row, for the tensor core's reads
            __syncwarp();
            if (lane == 0) mbar_arrive(p_full0 + 8 * s);
        }
        // ---- O / l -> bf16 -> global: each thread its 64 columns; l is the sum of the row's two partial sums ----
        if (!failed && nt > 0) {
            if (!mbar_wait(pv_done0 + 8 * ((nt - 1) & 1), ((nt - 1) >> 1) & 1)) { *sh_fail = 1; failed = true; }
            fence_after_sync();
        }
        asm volatile("bar.sync 2, 256;\n" ::: "memory");   // nobody still reads the last tile's maxima
        mx_s[wg * kT + r] = l_run;
        asm volatile("bar.sync 1, 256;\n" ::: "memory");
        const float l_row = l_run + mx_s[(wg ^ 1) * kT + r];
        if (n_split == 1) {
            __nv_bfloat16* orow = p.out + (size_t)(q_row0 + r) * 128 + wg * 64;
            const float inv = l_row > 0.f ? 1.f / l_row : 0.f;
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                uint32_t o[32];
                if (nt > 0 && !failed) {
                    tmem_ld32(lane_addr + kColO + wg * 64 + c * 32, o);
                    tmem_ld_wait();
                } else {
#pragma unroll
                    for (int k = 0; k < 32; ++k) o[k] = 0u;
                }
                if (row_ok) {
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        uint4 v;
                        v.x = pack2(__uint_as_float(o[8 * u]) * inv, __uint_as_float(o[8 * u + 1]) * inv);
                        v.y = pack2(__uint_as_float(o[8 * u + 2]) * inv, __uint_as_float(o[8 * u + 3]) * inv);
                        v.z = pack2(__uint_as_float(o[8 * u + 4]) * inv, __uint_as_float(o[8 * u + 5]) * inv);
                        v.w = pack2(__uint_as_float(o[8 * u + 6]) * inv, __uint_as_float(o[8 * u + 7]) * inv);
                        *reinterpret_cast<uint4*>(orow + c * 32 + u * 8) = v;
                    }
                }
            }
        } else {
            // this CTA's share of the keys: unnormalised O, m and l into its own shared memory (the K ring is spent)
            float* part_o = reinterpret_cast<float*>(smem + kSmK);      // [128 rows][32 float4], float4 index ^ (row & 31)
            float* part_ml = reinterpret_cast<float*>(smem + kSmV);     // [128] m, [128] l
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                uint32_t o[32];
                if (nt > 0 && !failed) {
                    tmem_ld32(lane_addr + kColO + wg * 64 + c * 32, o);
                    tmem_ld_wait();
                } else {
#pragma unroll
                    for (int k = 0; k < 32; ++k) o[k] = 0u;
                }
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    const int c4 = wg * 16 + c * 8 + u;
                    *reinterpret_cast<uint4*>(part_o + r * 128 + ((c4 ^ (r & 31)) << 2)) = make_uint4(o[4 * u], o[4 * u + 1], o[4 * u + 2], o[4 * u + 3]);
                }
            }
            if (wg == 0) { part_ml[r] = (nt > 0 && !failed) ? m_run : -INFINITY; part_ml[kT + r] = (nt > 0 && !failed) ? l_row : 0.f; }
        }
    }
    if (n_split > 1) {
        cg::cluster_group cluster = cg::this_cluster();
        fence_before_sync();
        cluster.sync();   // every member's partial is in its shared memory
        if (warp >= 2) {
            // this CTA folds query rows [split * R, (split + 1) * R) of the tile, R = 128 / n_split: one thread per
            // (row, four output columns), reading that piece of every member's partial
            const float* part_o = reinterpret_cast<const float*>(smem + kSmK);
            const float* part_ml = reinterpret_cast<const float*>(smem + kSmV);
            const int R = kT / n_split;
            for (int it = tid - 64; it < R * 32; it += 256) {
                const int r = split * R + (it >> 5), c4 = it & 31;
                float mv[kMaxSplit], lv[kMaxSplit];
                float4 ov[kMaxSplit];
#pragma unroll
                for (int j = 0; j < kMaxSplit; ++j) {
                    const int src = j < n_split ? j : 0;
                    const float* ml = cluster.map_shared_rank(part_ml, src);
                    const float* po = cluster.map_shared_rank(part_o, src);
                    mv[j] = j < n_split ? ml[r] : -INFINITY;
                    lv[j] = j < n_split ? ml[kT + r] : 0.f;
                    ov[j] = j < n_split ? *reinterpret_cast<const float4*>(po + r * 128 + ((c4 ^ (r & 31)) << 2)) : make_float4(0.f, 0.f, 0.f, 0.f);
                }
                float gm = mv[0];
#pragma unroll
                for (int j = 1; j < kMaxSplit; ++j) gm = fmaxf(gm, mv[j]);
                float lsum = 0.f;
                float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int j = 0; j < kMaxSplit; ++j) {
                    const float w = (mv[j] == -INFINITY) ? 0.f : ex2(mv[j] - gm);
                    lsum = fmaf(w, lv[j], lsum);
                    acc.x = fmaf(w, ov[j].x, acc.x); acc.y = fmaf(w, ov[j].y, acc.y);
                    acc.z = fmaf(w, ov[j].z, acc.z); acc.w = fmaf(w, ov[j].w, acc.w);
                }
                if (qt * kT + r < rows_total) {
                    const float inv = lsum > 0.f ? 1.f / lsum : 0.f;
                    uint2 v;
                    v.x = pack2(acc.x * inv, acc.y * inv);
                    v.y = pack2(acc.z * inv, acc.w * inv);
                    *reinterpret_cast<uint2*>(p.out + (size_t)(q_row0 + r) * 128 + c4 * 4) = v;
                }
            }
        }
        cluster.sync();   // every member's shared memory has been read: they may leave
    }
    __syncthreads();
    if (*sh_fail) {   // a wait gave up: report it and give copies still in flight one more bounded wait
        if (tid == 0) {
            set_status(p.status, SC_ERR_TIMEOUT);
            const int issued = *sh_issued;
            if (nt > 0) mbar_wait(q_full, 0);
            for (int t = max(issued - kStages, 0); t < issued; ++t) mbar_wait(kv_full0 + 8 * (t % kStages), (t / kStages) & 1);
        }
        __syncthreads();
    }
    fence_before_sync();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, kTmemCols);
}

// Any dtype, any d <= 256: one warp per (sequence, query head, query), online softmax in fp32.
template <typename T>
__global__ void __launch_bounds__(128) prefill_generic_kernel(const T* __restrict__ q, int B, int Hq, int Hkv, int m, int d,
                                                              const T* __restrict__ core_k, const T* __restrict__ core_v,
                                                              const int32_t* __restrict__ count, int cap,
                                                              const int32_t* __restrict__ core_len, float scale_log2, int causal,
                                                              T* __restrict__ out) {
    const int lane = threadIdx.x & 31;
    const long long it = (long long)blockIdx.x * 4 + (threadIdx.x >> 5);
    if (it >= (long long)B * Hq * m) return;
    const int i = (int)(it % m), hq = (int)((it / m) % Hq), b = (int)(it / ((long long)m * Hq));
    const int h = hq / (Hq / Hkv);
    const int len = max(min(core_len[b * Hkv + h], cap), 0);
    const int vis = causal ? len - (m - 1 - i) : len;
    const T* qr = q + it * d;
    const long long cbase = ((long long)b * Hkv + h) * cap;
    float qv[8], acc[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
        const int c = lane + 32 * u;
        qv[u] = c < d ? Elem<T>::load(qr + c) * scale_log2 : 0.f;
        acc[u] = 0.f;
    }
    float mx = -INFINITY, lsum = 0.f;
    for (int t = 0; t < vis; ++t) {
        const T* kr = core_k + (cbase + t) * d;
        const T* vr = core_v + (cbase + t) * d;
        float s = 0.f;
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int c = lane + 32 * u;
            if (c < d) s = fmaf(qv[u], Elem<T>::load(kr + c), s);
        }
        s = warp_sum(s);
        if (count != nullptr) s += log2f((float)max(count[cbase + t], 1));
        const float mn = fmaxf(mx, s);
        const float corr = exp2f(mx - mn), pw = exp2f(s - mn);
        lsum = lsum * corr + pw;
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int c = lane + 32 * u;
            if (c < d) acc[u] = acc[u] * corr + pw * Elem<T>::load(vr + c);
        }
        mx = mn;
    }
    const float inv = lsum > 0.f ? 1.f / lsum : 0.f;
#pragma unroll
    for (int u = 0; u < 8; ++u) {
        const int c = lane + 32 * u;
        if (c < d) Elem<T>::store(out + it * d + c, acc[u] * inv);
    }
}

}  // namespace pf

cudaError_t launch_prefill(const PrefillArgs& a, cudaStream_t st) {
    using namespace pf;
    const float scale_log2 = (a.scale == 0.f ? 1.f / sqrtf((float)a.d) : a.scale) * 1.4426950408889634f;
    const int causal = (a.flags & SC_FLAG_CAUSAL_TAIL) ? 1 : 0;
    const int G = a.Hq / a.Hkv;
    const long long q_rows = (long long)a.B * a.Hq * a.m, c_rows = (long long)a.B * a.Hkv * a.cap;
    if (a.dt == SC_BF16 && a.d == 128 && !(a.flags & SC_FLAG_GENERIC) && a.cap > 0 && q_rows < 0x7fffffff &&
        c_rows < 0x7fffffff && a.Hkv <= 65535 && a.B <= 65535) {
        // per device: the opt-in to large dynamic shared memory, the SM count, and the largest cluster of these
        // one-per-SM CTAs that can be scheduled
        static int sms_of[64] = {0}, cmax_of[64] = {0};
        int dev = 0;
        cudaGetDevice(&dev);
        dev &= 63;
        if (sms_of[dev] == 0) {
            cudaFuncSetAttribute(prefill_umma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
            int v = 0;
            cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev);
            int cmax = 1;
            for (int c = kMaxSplit; c > 1; c >>= 1) {
                cudaLaunchConfig_t probe = {};
                probe.gridDim = dim3(c, 1, 1);
                probe.blockDim = dim3(kThreads);
                probe.dynamicSmemBytes = kSmemBytes;
                cudaLaunchAttribute pa[1];
                pa[0].id = cudaLaunchAttributeClusterDimension;
                pa[0].val.clusterDim.x = c; pa[0].val.clusterDim.y = 1; pa[0].val.clusterDim.z = 1;
                probe.attrs = pa;
                probe.numAttrs = 1;
                int n_clusters = 0;
                if (cudaOccupancyMaxActiveClusters(&n_clusters, prefill_umma_kernel, &probe) == cudaSuccess && n_clusters > 0) {
                    cmax = c;
                    break;
                }
            }
            (void)cudaGetLastError();   // a refused probe is not an error of this call
            cmax_of[dev] = cmax;
            sms_of[dev] = v < 1 ? 1 : v;
        }
        Params p;
        p.count = a.count; p.core_len = a.core_len; p.out = (__nv_bfloat16*)a.out;
        p.Hq = a.Hq; p.Hkv = a.Hkv; p.m = a.m; p.cap = a.cap; p.causal = causal; p.scale_log2 = scale_log2; p.status = a.status;
        if (make_map_bf16_rows(&p.map_q, a.q, 0, 0, 128, 1, 1, q_rows, kT) &&
            make_map_bf16_rows(&p.map_k, a.core_k, 0, 0, 128, 1, 1, c_rows, kT) &&
            make_map_bf16_rows(&p.map_v, a.core_v, 0, 0, 128, 1, 1, c_rows, kT)) {
            // Few query tiles (short chunks, speculative decoding): split the keys over a cluster, as many ways as
            // fill the GPU, but leave every CTA at least two key tiles of the capacity.
            const long long ctas = (long long)((G * a.m + kT - 1) / kT) * a.Hkv * a.B;
            int n_split = 1;
            while (n_split * 2 <= cmax_of[dev] && ctas * n_split * 2 <= sms_of[dev] && (a.cap + kT - 1) / kT >= n_split * 4) n_split *= 2;
            p.n_split = n_split;
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3((unsigned)((G * a.m + kT - 1) / kT) * n_split, a.Hkv, a.B);
            cfg.blockDim = dim3(kThreads);
            cfg.dynamicSmemBytes = kSmemBytes;
            cfg.stream = st;
            cudaLaunchAttribute attr[1];
            attr[0].id = cudaLaunchAttributeClusterDimension;
            attr[0].val.clusterDim.x = n_split; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
            cfg.attrs = attr;
            cfg.numAttrs = 1;
            note_launches(1);
            return cudaLaunchKernelEx(&cfg, prefill_umma_kernel, p);
        }
    }
    const unsigned blocks = (unsigned)((q_rows + 3) / 4);
    if (a.dt == SC_BF16)
        prefill_generic_kernel<__nv_bfloat16><<<blocks, 128, 0, st>>>((const __nv_bfloat16*)a.q, a.B, a.Hq, a.Hkv, a.m, a.d,
            (const __nv_bfloat16*)a.core_k, (const __nv_bfloat16*)a.core_v, a.count, a.cap, a.core_len, scale_log2, causal,
            (__nv_bfloat16*)a.out);
    else
        prefill_generic_kernel<float><<<blocks, 128, 0, st>>>((const float*)a.q, a.B, a.Hq, a.Hkv, a.m, a.d, (const float*)a.core_k,
            (const float*)a.core_v, a.count, a.cap, a.core_len, scale_log2, causal, (float*)a.out);
    note_launches(1);
    return cudaGetLastError();
}

}  // namespace sc
