// Fused bf16 compress kernel (d = 128), sm_100a: Eq. 2 + Algorithm 1 + Eq. 3 in one pass over K, V.
//
// Persistent blocks (as many as fit on the GPU at once) draw work tiles from a global ticket
// counter.  A tile is a run of whole segments of at most SC_TILE_ROWS tokens of one (sequence, KV
// head) -- K and V both staged in shared memory -- or one longer segment alone (K staged, then V
// in a second pass over the same buffer).  Per tile:
//   1. the rows are staged by TMA (cp.async.bulk.tensor, boxes of 32 rows x 64 columns, 128-byte
//      swizzle so that ldmatrix is conflict free, completion on an mbarrier), issued by the block's
//      ninth "service" warp;
//   2. Eq. 2 + Algorithm 1, one warp per segment.  Up to 32 tokens (the usual case) everything
//      stays in registers: mma.m16n8k16 tiles laid over the segment's own rows give the upper
//      triangle of its Gram matrix (bf16 products are exact in fp32), the diagonal gives the norms,
//      Sim > tau is decided as G_ij > tau*|k_i|*|k_j|, each lane ends up with one row's adjacency
//      word, and the greedy pass costs one shuffle and a few word operations per seed;
//   3. the rows of segments of more than 32 tokens get their similarities from the tensor core: one thread issues
//      eight tcgen05.mma (128 x 128 x 128, bf16) on the staged rows -- the 128-byte-swizzled layout the TMA boxes
//      wrote is the K-major operand layout -- into tensor memory (three such blocks for a tile of 129..256 tokens,
//      the diagonal ones first: they give the norms); the warps that own such rows read the accumulator one row per
//      thread and keep, as bits in registers, which EARLIER tokens of its segment each row is similar to.
//      Algorithm 1 is then settled for all those rows at once, in rounds: a row with an earlier neighbour that is
//      a seed is a member, a row whose earlier neighbours are all members is a seed (the lowest open row is decided
//      in every round, so the rounds end; chunks that are unions of cliques take two).  A member joins the earliest
//      seed among its neighbours, which is what the sequential pass does; the lanes of a warp that name the same
//      seed are found with match.any and write that word of the seed's member mask.  Warps without such rows do
//      the short segments meanwhile (segments are claimed from a counter, not dealt by warp number);
//   4. the tile's cluster count enters a prefix sum over the tiles of its (sequence, head): a
//      decoupled look-back over per-tile status words (tickets are handed out in order, so every
//      predecessor is held by a running block and the bounded wait cannot starve), or, in
//      two-pass mode, a count pass followed by a write pass;
//   5. Eq. 3, beside the service warp's look-back: every token belongs to exactly one cluster, so a
//      cluster's mean can overwrite its seed's staged row.  The clusters are dealt to the compute
//      warps in seed order; a lane owns eight columns of the K or of the V row, sums the member
//      rows in fp32 in token order, scales by 1/|S| and rounds once to bf16; clusters of one token
//      are left as they are.  The cores then leave in seed order with 16-byte coalesced stores.
//      The service warp draws the block's next ticket during step 2.
// The last block to finish zeroes the status words and counters, so a workspace that was zero
// before the call is zero again after it.
// One launch may serve several layers (sc_compress_layers): the tickets then go round the (layer, sequence,
// head) units, which puts L*B*Hkv tickets between consecutive tiles of a head instead of B*Hkv; with few heads
// per layer that is what keeps one late tile from holding up every tile of its head that is in flight.
#include <cuda.h>

#include <mutex>

#include "common.cuh"
#include "umma.cuh"

namespace sc {

namespace cf {

constexpr int kWarps = 8;                         // compute warps
constexpr int kThreads = (kWarps + 1) * 32;       // plus one service warp: next ticket, look-back
constexpr int kD = 128;
constexpr int kRowBytes = 256;                    // one K or V row in global memory
constexpr int kHalfRow = 128;                     // a staged row is two 128-byte halves (64 columns each), see tile_addr
constexpr int kBoxRows = 32;                      // rows per TMA box
constexpr int kBoxBytes = kBoxRows * kHalfRow;    // 4096
constexpr int kMaxRows = SC_MAX_CHUNK_LEN;        // 256: a long tile
constexpr int kShortRows = SC_TILE_ROWS;          // 128
// Longest segment one warp clusters on its own, in registers; the bit rows of longer ones come from the tile's Gram
// matrix on the tensor core.  (A warp-private mma.sync path for 33..48 tokens was 16 % slower on lognormal chunks.)
constexpr int kWarpSegMax = 32;
constexpr int kNW = 8;                            // 32-bit words per (full) adjacency row
constexpr int kKvBytes = kMaxRows * kRowBytes;    // 65536: short = K | V, long = one tensor
constexpr int kVOff = kShortRows * kRowBytes;     // 32768
constexpr int kHalfShort = kShortRows * kHalfRow; // 16384: distance between the column halves of a short tile
constexpr int kHalfLong = kMaxRows * kHalfRow;    // 32768: ... of a long one
constexpr int kCntOff = kKvBytes;                 // uint32[256] per seed row: what pool_clusters needs, then the member count
constexpr int kAdjOff = kCntOff + kMaxRows * 4;
constexpr int kAdjWords = 32 * (8 + 7 + 6 + 5 + 4 + 3 + 2 + 1);   // rows of block k keep words k..7
constexpr int kNormOff = kAdjOff + kAdjWords * 4; // float[512]: norms (64 per warp, or one per row); later uint16 seed row per cluster
constexpr int kRowNormOff = kNormOff + kWarps * 64 * 4; // float[256]: norms of the rows of long segments (from the tensor core's Gram diagonal)
constexpr int kSegsOff = kRowNormOff + kMaxRows * 4; // 2 x int16[132]: segment starts (this tile, next tile)
constexpr int kSegsStride = 132;
constexpr int kMiscOff = kSegsOff + 2 * kSegsStride * 2;   // uint32 seedmask[8]; int geo[2][8]; int misc[4]
constexpr int kBarOff = kMiscOff + 32 + 64 + 16 + 32 + 128 + 16 + 32;   // ... 8 spare words; uint8 multi[128]; tensor-memory slot, flag; uint32 membits[8]; three mbarriers
constexpr int kSmemBytes = kBarOff + 24;
constexpr int kTmemCols = 128;                    // one 128 x 128 fp32 accumulator per block (three blocks per SM: 384 of 512 columns)
constexpr int kBlocksPerSm = 3;
static_assert(kBarOff % 8 == 0, "mbarrier alignment");
static_assert(kSmemBytes <= 76800, "three blocks per SM need <= 75 KB each");

enum Mode { kCountOnly = 0, kWriteWithCounts = 1, kLookBack = 2 };
enum Geo { gB = 0, gH = 1, gT = 2, gNseg = 3, gRow0 = 4, gR = 5, gLast = 6, gLayer = 7 };

// cnts[seed row] while the cluster waits to be pooled: kPending | first row of its segment | (one past its last
// row) << 9, the latter 0 for a segment of up to 32 tokens, whose member mask is one segment-relative word
constexpr uint32_t kPending = 1u << 31;
constexpr uint32_t kFlagAggregate = 1u << 30, kFlagPrefix = 2u << 30, kValueMask = (1u << 30) - 1;
constexpr unsigned long long kWaitLimitNs = 2000000000ull;   // every wait gives up after 2 s
constexpr int kPollGroups = 2;                               // the look-back reads 64 predecessors per poll (4 and 8 measured slower, 1 slower on short chunks)
constexpr int kCtlWords = 64;                                // ticket, done counter, padding

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;\n" : "=l"(t));
    return t;
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}\n"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0u;
}
// Bounded wait for a phase of an mbarrier; false if it gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_ns();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 256; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (global_ns() - t0 > kWaitLimitNs) return false;
    }
}
// One TMA box: 32 rows x 64 columns of a [B, Hkv, n, 128] tensor, 128-byte swizzled, no multicast.
__device__ __forceinline__ void tma_box(uint32_t dst, const CUtensorMap* map, int col, int row, int h, int b, uint32_t bar) {
    asm volatile("cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];\n"
                 ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(col), "r"(row), "r"(h), "r"(b), "r"(bar) : "memory");
}
__device__ __forceinline__ void fence_async_proxy() { asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory"); }
// Byte offset, inside one column half of a staged tensor, of 16-byte chunk `chunk` (0..7) of row
// `row`: rows are 128 bytes apart and the chunk index is XORed with the row's low three bits (the
// TMA 128-byte swizzle), which makes ldmatrix over eight consecutive rows conflict free.
__device__ __forceinline__ uint32_t tile_addr(int row, int chunk) { return row * kHalfRow + ((chunk ^ (row & 7)) << 4); }
__device__ __forceinline__ void compute_warps_sync() {   // the eight compute warps, not the service warp
    asm volatile("bar.sync 1, 256;\n" ::: "memory");
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
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
// Word offset of adjacency word (row i, word i>>5) in the triangular store; word w >= i>>5 of the
// same row follows at + (w - (i>>5)).
__device__ __forceinline__ int adj_row(int i) {
    const int k = i >> 5;
    return 256 * k - 16 * k * (k - 1) + (i & 31) * (kNW - k);
}

// 16 consecutive fp32 columns of this thread's tensor-memory lane.
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];\n"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr) : "memory");
}

// One 128 x 128 block of K.K^T of the staged keys: rows of 128-row block mb against rows of block nb (column
// halves `hs` bytes apart, 128-byte-swizzled rows: what the TMA boxes wrote is the K-major layout tcgen05.mma
// reads).  One thread issues the eight instructions; the mbarrier gets one arrival when they are complete.
__device__ __forceinline__ void umma_gram_block(uint32_t kbase, int hs, int mb, int nb, uint32_t tmem, uint32_t bar) {
    constexpr uint32_t idesc = umma::instr_desc_bf16(128, 128, false, false);
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
        const uint32_t off = (ks >> 2) * hs + (ks & 3) * 32;
        umma::mma_bf16_ss(tmem, umma::smem_desc_sw128(kbase + mb * 128 * kHalfRow + off, 16, 1024),
                          umma::smem_desc_sw128(kbase + nb * 128 * kHalfRow + off, 16, 1024), idesc, ks > 0);
    }
    umma::mma_commit(bar);
}

// The diagonal of a diagonal block = squared norms: thread (quarter q, lane) of the four reading warps owns tile
// row mb*128 + 32q + lane and finds its element in the 32 columns its warp's rows share.
__device__ __forceinline__ void umma_norms(uint32_t tmem, int mb, int q, int lane, float* norm) {
    const uint32_t lane_addr = tmem + ((uint32_t)(q * 32) << 16);
    float v = 0.f;
#pragma unroll
    for (int c = 0; c < 2; ++c) {
        uint32_t g[16];
        tmem_ld16(lane_addr + q * 32 + c * 16, g);
        umma::tmem_ld_wait();
#pragma unroll
        for (int k = 0; k < 16; ++k)
            if (lane == c * 16 + k) v = __uint_as_float(g[k]);
    }
    norm[mb * 128 + q * 32 + lane] = sqrtf(v);
}

// Reads this thread's row i = 128 mb + 32 q + lane of the block in tensor memory and returns, as four words over
// the block's columns 128 nb .. 128 nb + 127, which EARLIER tokens of i's own segment [a_i, ...) are similar to it:
// bit c of the result = Sim(c, i) > tau for a_i <= c < i, decided as G > |k_c| (tau |k_i|) -- the earlier token's
// norm first, the product the short-segment path forms for the same pair.  Only the chunks of sixteen columns
// that can hold a column below the warp's rows are read (`chunks`), and no word before the first (`w_lo`) that
// holds a token of a segment one of the warp's rows is in (both uniform over the warp).
template <bool kNegTau>
__device__ __forceinline__ void umma_earlier(uint32_t tmem, int nb, int q, int i, int a_i, float tau, const float* norm,
                                             int w_lo, int chunks, uint32_t (&words)[4]) {
    const uint32_t lane_addr = tmem + ((uint32_t)(q * 32) << 16);
    const float tni = tau * norm[i];
#pragma unroll
    for (int c = 0; c < 4; ++c) {   // 32 columns = one word at a time
        uint32_t w = 0u;
        if (c >= w_lo && 2 * c < chunks) {   // a word that holds an earlier token of some row's segment
            uint32_t g[32];
            umma::tmem_ld32(lane_addr + c * 32, g);
            umma::tmem_ld_wait();
            const float4* nc = reinterpret_cast<const float4*>(norm + nb * 128 + c * 32);
#pragma unroll
            for (int k4 = 0; k4 < 8; ++k4) {
                const float4 nv = nc[k4];
                const float thr[4] = {nv.x * tni, nv.y * tni, nv.z * tni, nv.w * tni};
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    bool hit = __uint_as_float(g[k4 * 4 + k]) > thr[k];
                    if (kNegTau) hit = hit || (thr[k] == 0.f);   // a zero-norm key has Sim = 0 > tau
                    w |= (hit ? 1u : 0u) << (k4 * 4 + k);
                }
            }
        }
        words[c] = w & bits_between(a_i, i, nb * 4 + c);
    }
}

// One round of Algorithm 1's decisions for the 32 tokens a warp owns (tile word `word`, token 32 word + lane),
// on each token's earlier-neighbour words `e`: a token with an earlier neighbour that is a seed is a member; a
// token whose earlier neighbours are all members is a seed.  Both facts are final once true, so reading words
// that other warps are updating is harmless.  `open` = not yet decided (false for tokens outside long segments);
// the warp's new seeds and members go to the shared words with one atomic each.
__device__ __forceinline__ void decide_round(const uint32_t (&e)[8], int word, int lane, bool& open, bool& is_seed,
                                             volatile uint32_t* seeds, volatile uint32_t* members) {
    // all lanes read the same sixteen words (broadcast), no branch per word
    uint32_t sd[8], mb[8];
#pragma unroll
    for (int w = 0; w < 8; ++w) { sd[w] = seeds[w]; mb[w] = members[w]; }
    uint32_t near_seed = 0u, not_member = 0u;
#pragma unroll
    for (int w = 0; w < 8; ++w) { near_seed |= e[w] & sd[w]; not_member |= e[w] & ~mb[w]; }
    const bool to_member = open && near_seed != 0u;
    const bool to_seed = open && near_seed == 0u && not_member == 0u;
    if (to_member || to_seed) open = false;
    if (to_seed) is_seed = true;
    const uint32_t nm = __ballot_sync(kFull, to_member), ns = __ballot_sync(kFull, to_seed);
    if (lane == 0) {
        if (nm) atomicOr(const_cast<uint32_t*>(members) + word, nm);
        if (ns) atomicOr(const_cast<uint32_t*>(seeds) + word, ns);
    }
}

// After the rounds: a member joins the earliest seed among its earlier neighbours, as Algorithm 1 would have it.
// The lanes of a warp that name the same seed are that cluster's members in the warp's word: one of them writes
// the word into the seed's row of the triangular store (the seed's member mask, tile positions; the seed itself
// is in it).  Words of the row that get no member were cleared beforehand.
__device__ __forceinline__ void settle_round(const uint32_t (&e)[8], int word, int lane, bool active, bool is_seed,
                                             int a_i, int e_i, const volatile uint32_t* seeds, uint32_t* adj,
                                             uint32_t* cnts, int32_t* as, int row0) {
    const int i = word * 32 + lane;
    int s = active ? i : -1 - lane;   // inactive lanes: keys of their own
    if (active && !is_seed) {
#pragma unroll
        for (int w = 7; w >= 0; --w) {
            const uint32_t m = e[w] & seeds[w];
            if (m) s = w * 32 + __ffs(m) - 1;
        }
    }
    const uint32_t group = __match_any_sync(kFull, s);
    if (!active) return;
    if (is_seed) cnts[i] = kPending | (uint32_t)a_i | ((uint32_t)e_i << 9);
    if ((int)(__ffs(group) - 1) == lane) adj[adj_row(s) + word - (s >> 5)] = group;
    if (as) as[i] = row0 + s;
}

// `threads` threads of the block (whole warps) meet at barrier 2 ...
__device__ __forceinline__ void warps_sync(int threads) { asm volatile("barrier.cta.sync 2, %0;\n" ::"r"(threads) : "memory"); }
// ... and learn whether any of them still has work.
__device__ __forceinline__ bool warps_any(bool mine, int threads) {
    uint32_t out;
    asm volatile(
        "{\n"
        ".reg .pred p, r;\n"
        "setp.ne.u32 p, %1, 0;\n"
        "barrier.cta.red.or.pred r, 2, %2, p;\n"
        "selp.u32 %0, 1, 0, r;\n"
        "}\n"
        : "=r"(out) : "r"(mine ? 1u : 0u), "r"(threads) : "memory");
    return out != 0u;
}

// Step 2 for one tile: Algorithm 1 for the rows of segments of more than kWarpSegMax tokens (all threads of the
// block call it; a wait for the tensor core that gave up is left in the tile's failure flag).  The Gram matrix comes
// from the tensor core, 128 x 128 at a time into tensor memory: one block for a tile of up to 128 tokens, else the
// two diagonal blocks -- they give the norms -- and the lower one.  Compute thread tid settles tile row tid: warps
// 0..3 read the accumulator rows of block 0, warps 4..7 those of block 1 (a warp reaches the tensor-memory lanes of
// its quarter, warp % 4), and keep which earlier tokens of its segment each row is similar to; Algorithm 1 is then
// settled for all those rows at once in decision rounds.  `words` has a bit for every 32-row word of the tile that
// a long segment touches: in a tile of up to 128 rows only those warps stay, the others (and the service warp, once
// it has issued the product) leave at once for the short segments and the next ticket.  Kept out of line: its
// registers are not the main loop's.
__device__ __noinline__ void settle_long_segments(unsigned char* smem, int hs, const int16_t* segs, int nseg, int R,
                                                  uint32_t words, uint32_t tmem, uint32_t phase_u, float tau,
                                                  int32_t* as, int row0) {
    uint32_t* cnts = reinterpret_cast<uint32_t*>(smem + kCntOff);
    uint32_t* adj = reinterpret_cast<uint32_t*>(smem + kAdjOff);
    float* norm = reinterpret_cast<float*>(smem + kRowNormOff);
    uint32_t* seedmask = reinterpret_cast<uint32_t*>(smem + kMiscOff);
    volatile int* umma_failed = reinterpret_cast<volatile int*>(smem + kMiscOff + 276);
    uint32_t* membits = reinterpret_cast<uint32_t*>(smem + kMiscOff + 288);
    const uint32_t sbase = smem_u32(smem), bar_u = sbase + kBarOff + 16;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, q = warp & 3;
    const bool service = warp == kWarps;
    const bool long_tile = R > kShortRows;
    if (!long_tile) {
        if (service) {
            if (lane == 0) {
                umma::fence_after_sync();
                umma_gram_block(sbase, hs, 0, 0, tmem, bar_u);
            }
            return;
        }
        if (!((words >> warp) & 1u)) return;
    }
    const int team = long_tile ? kWarps * 32 : 32 * __popc(words & 0xffu);   // threads that meet at barrier 2
    // the segment [beg, end) this thread's row is in: the last start that is not beyond the row
    int beg = tid, end = tid;
    if (tid < R) {
        int lo = 0, hi = nseg;   // segs[lo] <= tid < segs[hi]
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if ((int)segs[mid] <= tid) lo = mid; else hi = mid;
        }
        beg = segs[lo]; end = segs[hi];
    }
    const bool act = end - beg > kWarpSegMax;   // rows of shorter segments take no part
    uint32_t ern[8] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u};   // earlier neighbours of the row, tile words
    if (!long_tile) {
        if (!mbar_wait(bar_u, phase_u)) *umma_failed = 1;   // carry on (the barriers below must be met); the tile is dropped later
        umma::fence_after_sync();
        umma_norms(tmem, 0, q, lane, norm);
        warps_sync(team);   // the norms of every row of a long segment are in place
        uint32_t w4[4];
        const int w_lo = __reduce_min_sync(kFull, act ? beg >> 5 : kNW);   // first word any of the warp's rows needs
        if (tau < 0.f) umma_earlier<true>(tmem, 0, q, tid, beg, tau, norm, w_lo, 2 * q + 2, w4);
        else umma_earlier<false>(tmem, 0, q, tid, beg, tau, norm, w_lo, 2 * q + 2, w4);
        ern[0] = w4[0]; ern[1] = w4[1]; ern[2] = w4[2]; ern[3] = w4[3];
        umma::fence_before_sync();
    } else {
        for (int ps = 0; ps < 3; ++ps) {   // (0,0); (1,1), (1,0)
            const int mb = ps == 0 ? 0 : 1, nb = ps == 1 ? 1 : 0;
            const bool reader = !service && (warp >> 2) == mb;
            if (service && lane == 0) {
                umma::fence_after_sync();
                umma_gram_block(sbase, hs, mb, nb, tmem, bar_u);
            }
            if (reader) {
                if (!mbar_wait(bar_u, phase_u)) *umma_failed = 1;
                umma::fence_after_sync();
                if (mb == nb) umma_norms(tmem, mb, q, lane, norm);
            }
            phase_u ^= 1u;
            __syncthreads();   // the norms are in place
            if (reader) {
                const int chunks = mb == nb ? 2 * q + 2 : 8;   // a diagonal block: columns below the warp's rows
                uint32_t w4[4];
                if (tau < 0.f) umma_earlier<true>(tmem, nb, q, tid, beg, tau, norm, 0, chunks, w4);
                else umma_earlier<false>(tmem, nb, q, tid, beg, tau, norm, 0, chunks, w4);
                if (nb == 0) { ern[0] = w4[0]; ern[1] = w4[1]; ern[2] = w4[2]; ern[3] = w4[3]; }
                else { ern[4] = w4[0]; ern[5] = w4[1]; ern[6] = w4[2]; ern[7] = w4[3]; }
                umma::fence_before_sync();
            }
            if (ps < 2) __syncthreads();   // the accumulator may be overwritten
        }
        if (service) return;
    }
    // the row's place in the triangular store will hold the member mask if the row is a seed
    if (act) for (int ww = warp; ww <= (end - 1) >> 5; ++ww) adj[adj_row(tid) + ww - warp] = 0u;
    bool open = act, is_seed = false;
    do {
        decide_round(ern, warp, lane, open, is_seed, seedmask, membits);
    } while (warps_any(open, team));   // the lowest open token is decided every round
    settle_round(ern, warp, lane, act, is_seed, beg, end, seedmask, adj, cnts, as, row0);
}

// Eq. 3 building blocks.  A lane owns eight consecutive columns (one 16-byte chunk) of the K row
// (lanes 0-15) or of the V row (lanes 16-31); `lane_base` is its tensor and column half, c7 its
// chunk inside the half.  Sums are fp32, in token order.
// s0 += low bf16 of v, s1 += high bf16 of v: the mixed-precision add takes the bf16 operand as it is (exact
// widening, one fp32 rounding of the sum -- what unpacking by hand and adding gives, in half the instructions).
__device__ __forceinline__ void add_pair(uint32_t v, float& s0, float& s1) {
    asm("{\n.reg .b16 lo, hi;\nmov.b32 {lo, hi}, %2;\nadd.rn.f32.bf16 %0, lo, %0;\nadd.rn.f32.bf16 %1, hi, %1;\n}\n"
        : "+f"(s0), "+f"(s1) : "r"(v));
}
__device__ __forceinline__ void add_chunk(const uint4& v, float (&s)[8]) {
    add_pair(v.x, s[0], s[1]);
    add_pair(v.y, s[2], s[3]);
    add_pair(v.z, s[4], s[5]);
    add_pair(v.w, s[6], s[7]);
}
// Adds the rows first + j for every set bit j of mem, in order; two loads are kept in flight (the
// filler of an odd count is a row of zeros, which leaves the sums as they are).
__device__ __forceinline__ void rows_add(const unsigned char* lane_base, int first, uint32_t mem, int c7, float (&s)[8]) {
    while (mem) {
        const int j0 = __ffs(mem) - 1;
        mem &= mem - 1;
        const uint4 v0 = *reinterpret_cast<const uint4*>(lane_base + tile_addr(first + j0, c7));
        uint4 v1 = make_uint4(0u, 0u, 0u, 0u);
        if (mem) {
            const int j1 = __ffs(mem) - 1;
            mem &= mem - 1;
            v1 = *reinterpret_cast<const uint4*>(lane_base + tile_addr(first + j1, c7));
        }
        add_chunk(v0, s);
        add_chunk(v1, s);
    }
}
__device__ __forceinline__ void row_put_mean(unsigned char* lane_base, int row, int c7, const float (&s)[8], float inv) {
    __nv_bfloat162 a = __floats2bfloat162_rn(s[0] * inv, s[1] * inv), b = __floats2bfloat162_rn(s[2] * inv, s[3] * inv);
    __nv_bfloat162 c = __floats2bfloat162_rn(s[4] * inv, s[5] * inv), d = __floats2bfloat162_rn(s[6] * inv, s[7] * inv);
    uint4 v;
    v.x = *reinterpret_cast<uint32_t*>(&a); v.y = *reinterpret_cast<uint32_t*>(&b);
    v.z = *reinterpret_cast<uint32_t*>(&c); v.w = *reinterpret_cast<uint32_t*>(&d);
    *reinterpret_cast<uint4*>(lane_base + tile_addr(row, c7)) = v;
}

// Eq. 2 + Algorithm 1 for one segment of 2..32 tokens, by one warp, in registers.
// Rows [a, a + l) of the staged keys.  The upper triangle of the segment's own Gram matrix comes
// from mma tiles laid over the segment's rows (16-row tiles down, 8-column tiles across, only
// those that reach above the diagonal); lane 4g + t ends up owning row g + 8t with its adjacency
// bits (later tokens only) in one word, and the greedy pass is a handful of word operations and
// one shuffle per seed.  Results: seed bits into the tile's seedmask; for pool_clusters each seed's
// member mask (bit j = token a + j) in the first word of its adjacency row and a note in cnts;
// optionally the seed of every token.
template <bool kNegTau>
__device__ __forceinline__ void gsc_short_segment(uint32_t kbase, int hs, int a, int l, float tau, float* nrm /*[32], this warp's*/,
                                                  uint32_t* seedmask, uint32_t* adj, uint32_t* cnts, int32_t* as, int row0,
                                                  int lane) {
    const int g = lane >> 2, tig = lane & 3;
    const int nnt = (l + 7) >> 3;          // 8-column tiles that hold tokens: 1..4
    const bool two_mt = l > 16;
    float acc[2][4][4];
#pragma unroll
    for (int mt = 0; mt < 2; ++mt)
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) acc[mt][nt][0] = acc[mt][nt][1] = acc[mt][nt][2] = acc[mt][nt][3] = 0.f;
    {
        const int j = lane >> 3, r8 = lane & 7;
        const uint32_t a_base = kbase + tile_addr(a + r8 + ((j & 1) << 3), j >> 1);
        const uint32_t b_base = kbase + tile_addr(a + r8 + ((j >> 1) << 3), j & 1);
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
            uint32_t a0[4], a1[4], b0[4], b1[4];
            const uint32_t a_addr = (a_base ^ ((ks & 3) << 5)) + (ks >> 2) * hs;
            const uint32_t b_addr = (b_base ^ ((ks & 3) << 5)) + (ks >> 2) * hs;
            ldmatrix_x4(a_addr, a0[0], a0[1], a0[2], a0[3]);
            ldmatrix_x4(b_addr, b0[0], b0[1], b0[2], b0[3]);
            mma_bf16(acc[0][0], a0[0], a0[1], a0[2], a0[3], b0[0], b0[1]);
            if (nnt > 1) mma_bf16(acc[0][1], a0[0], a0[1], a0[2], a0[3], b0[2], b0[3]);
            if (two_mt) {
                ldmatrix_x4(a_addr + 16 * kHalfRow, a1[0], a1[1], a1[2], a1[3]);
                ldmatrix_x4(b_addr + 16 * kHalfRow, b1[0], b1[1], b1[2], b1[3]);
                mma_bf16(acc[0][2], a0[0], a0[1], a0[2], a0[3], b1[0], b1[1]);
                mma_bf16(acc[1][2], a1[0], a1[1], a1[2], a1[3], b1[0], b1[1]);
                if (nnt > 3) {
                    mma_bf16(acc[0][3], a0[0], a0[1], a0[2], a0[3], b1[2], b1[3]);
                    mma_bf16(acc[1][3], a1[0], a1[1], a1[2], a1[3], b1[2], b1[3]);
                }
            }
        }
    }
    // norms from the diagonal
    if ((g >> 1) == tig) {
        const int e = g & 1;
#pragma unroll
        for (int mt = 0; mt < 2; ++mt)
#pragma unroll
            for (int hh = 0; hh < 2; ++hh)
                nrm[mt * 16 + hh * 8 + g] = sqrtf(e ? acc[mt][2 * mt + hh][hh * 2 + 1] : acc[mt][2 * mt + hh][hh * 2]);
    }
    __syncwarp();
    float tn[4][2];
#pragma unroll
    for (int nt = 0; nt < 4; ++nt) {
        const float2 nn = *reinterpret_cast<const float2*>(nrm + nt * 8 + 2 * tig);
        tn[nt][0] = tau * nn.x;
        tn[nt][1] = tau * nn.y;
    }
    uint32_t wrow[2][2];
#pragma unroll
    for (int mt = 0; mt < 2; ++mt)
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
            uint32_t w = 0;
            if (mt == 0 || two_mt) {
                const float ni = nrm[mt * 16 + hh * 8 + g];
#pragma unroll
                for (int nt = 0; nt < 4; ++nt) {
                    if (nt < 2 * mt + hh) continue;   // columns before the row's own
                    if (nt < nnt) {
#pragma unroll
                        for (int e = 0; e < 2; ++e) {
                            const float thr = ni * tn[nt][e];
                            bool hit = acc[mt][nt][hh * 2 + e] > thr;
                            if (kNegTau) hit = hit || (thr == 0.f);   // a zero-norm key has Sim = 0 > tau
                            if (hit) w |= 1u << (nt * 8 + e);
                        }
                    }
                }
                w <<= 2 * tig;
                w |= __shfl_xor_sync(kFull, w, 1);
                w |= __shfl_xor_sync(kFull, w, 2);
            }
            wrow[mt][hh] = w;
        }
    __syncwarp();   // the norms are spent: the next segment of this warp may overwrite them
    // lane 4g + t owns token g + 8t
    const int own = g + 8 * tig;
    const uint32_t lowmask = l >= 32 ? 0xffffffffu : ((1u << l) - 1u);
    uint32_t mine = (tig & 2) ? ((tig & 1) ? wrow[1][1] : wrow[1][0]) : ((tig & 1) ? wrow[0][1] : wrow[0][0]);
    mine &= (0xfffffffeu << own) & lowmask;   // later tokens of the segment only
    // Algorithm 1
    uint32_t U = lowmask, seeds = 0u, mymem = 0u;
    int seed_of = 0;
    while (U) {
        const int i = __ffs(U) - 1;                      // lowest unassigned token: a seed
        const int src = ((i & 7) << 2) | (i >> 3);
        const uint32_t mem = (__shfl_sync(kFull, mine, src) & U) | (1u << i);
        U &= ~mem;
        if ((mem >> own) & 1u) seed_of = i;
        if (lane == src) mymem = mem;
        seeds |= 1u << i;
    }
    // hand the result to the tile
    const int sh = a & 31, w0 = a >> 5;
    if (lane == 0) {
        atomicOr(&seedmask[w0], seeds << sh);
        if (sh != 0 && (seeds >> (32 - sh)) != 0u) atomicOr(&seedmask[w0 + 1], seeds >> (32 - sh));
    }
    if (mymem != 0u) {
        adj[adj_row(a + own)] = mymem;
        cnts[a + own] = kPending | (uint32_t)a;
    }
    if (as != nullptr && own < l) as[a + own] = row0 + a + seed_of;
}

// Eq. 3 for the tile's P clusters (seedrow[c] = seed row of cluster c), dealt to the compute warps in turn.  Every token belongs to
// exactly one cluster, so a cluster's mean can overwrite its seed's staged row once its members are
// summed (fp32, token order); a cluster of one is left as it is.  cnts[seed row] ends up holding the
// member count.  `lanes` is 32 when K and V are both staged, 16 when only K is.
__device__ __forceinline__ void pool_clusters(unsigned char* lane_base, const uint16_t* seedrow, int P, const uint32_t* adj,
                                              uint32_t* cnts, int warp, int lane, int lanes) {
    const int c7 = lane & 7;
    {
        for (int c = warp; c < P; c += kWarps) {
            const int i = seedrow[c];
            const uint32_t info = cnts[i];
            if (!(info & kPending)) continue;   // a one-token segment: settled when the tile was staged
            const int a = info & 511, e = (info >> 9) & 511;
            float sum[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
            int cnt;
            if (e == 0) {   // up to 32 tokens: one word, relative to the segment
                uint32_t mem = adj[adj_row(i)];
                cnt = __popc(mem);
                if (cnt > 1 && lane < lanes) rows_add(lane_base, a, mem, c7, sum);
            } else {        // longer: the row's words, at tile positions
                const uint32_t* row = adj + adj_row(i) - (i >> 5);
                cnt = 0;
                for (int ww = i >> 5; ww <= (e - 1) >> 5; ++ww) {
                    const uint32_t mem = row[ww];
                    cnt += __popc(mem);
                    if (lane < lanes) rows_add(lane_base, ww * 32, mem, c7, sum);
                }
            }
            __syncwarp();
            if (lane == 0) cnts[i] = (uint32_t)cnt;
            if (cnt > 1 && lane < lanes) row_put_mean(lane_base, i, c7, sum, 1.0f / (float)cnt);
        }
    }
}

// What differs between the layers of a multi-layer launch (sc_compress_layers); a one-layer launch has one.
struct LayerRefs {
    CUtensorMap map_k, map_v;   // [B, Hkv, n, 128] bf16, boxes of 32 rows x 64 columns, 128-byte swizzle
    __nv_bfloat16* core_k; __nv_bfloat16* core_v; int32_t* count; int32_t* core_len; int32_t* assign;
};
constexpr int kMaxLayers = 64;   // layers per launch (the launch parameters hold their tensor maps)

template <int NL>
struct Params {
    int B, Hkv, n, L;
    const int32_t* seg_off; const int32_t* tile_seg; const int32_t* seq_tile_cnt; int n_tile_cap;
    float tau;
    int cap;
    int32_t* ctl;            // [0] ticket counter, [1] blocks finished
    uint32_t* tile_state;    // [L][B*Hkv][n_tile_cap]
    int32_t* status;
    const float* tau_dev;    // threshold in device memory (budget search), or null: use tau
    const int32_t* skip;     // device flag: nonzero = this launch has nothing to do (budget search), or null
    int count_into_len;      // kCountOnly: add the tile's cluster count to core_len instead of recording it per tile
    LayerRefs layer[NL];
};



// The service warp draws the next ticket, turns it into a tile (sequence, head, tile index, rows) and
// copies the tile's segment starts into shared memory.  Tickets go round the (sequence, head) pairs:
// ticket w is tile w / (B*Hkv) of pair w % (B*Hkv), so consecutive tiles of one head are B*Hkv
// tickets apart and a tile's predecessor has usually published its cluster count (and often its
// prefix) by the time the tile looks back.  A pair with fewer tiles skips its surplus tickets.
// geo[gT] = -1 when no work is left (max_nt = most tiles any sequence has).
template <int NL>
__device__ __forceinline__ void fetch_tile(const Params<NL>& p, int lane, int max_nt, int* geo, int16_t* segs) {
    const int pairs = p.B * p.Hkv, units = pairs * p.L;   // (layer, sequence, head) units take the tickets in turn
    int b, h, t, nt, ly;
    for (;;) {
        int w = 0;
        if (lane == 0) w = atomicAdd(&p.ctl[0], 1);
        w = __shfl_sync(kFull, w, 0);
        t = w / units;
        if (t >= max_nt) {
            if (lane == 0) geo[gT] = -1;
            return;
        }
        const int unit = w - t * units;
        ly = unit / pairs;
        const int bh = unit - ly * pairs;
        b = bh / p.Hkv;
        h = bh - b * p.Hkv;
        nt = min(p.seq_tile_cnt[b], p.n_tile_cap);
        if (t < nt) break;
    }
    const int32_t* ts = p.tile_seg + (size_t)b * (p.n_tile_cap + 1);
    const int s_begin = ts[t], s_end = ts[t + 1];
    const int nseg = max(min(s_end - s_begin, kShortRows), 1);
    const int g_row0 = p.seg_off[s_begin];
    for (int i = lane; i <= nseg; i += 32) segs[i] = (int16_t)min(p.seg_off[s_begin + i] - g_row0, kMaxRows);
    const int R = min(p.seg_off[s_begin + nseg] - g_row0, kMaxRows);
    if (lane == 0) {
        geo[gB] = b; geo[gH] = h; geo[gT] = t; geo[gNseg] = nseg; geo[gRow0] = g_row0 - b * p.n; geo[gR] = R;
        geo[gLast] = (t == nt - 1);
        geo[gLayer] = ly;
    }
}

// Stages rows [row0, row0 + R) of head (b, h) of one tensor with TMA: one box of 32 rows x 64 columns
// per lane (R <= 256 needs at most 16 boxes for both column halves), the halves `hs` bytes apart at
// `dst`.  Rows past R inside the last box are the cache's next rows, or zeros past the end of the
// sequence; no one reads them.
__device__ __forceinline__ void stage_rows(uint32_t dst, int hs, const CUtensorMap* map, int row0, int R, int h, int b,
                                           uint32_t bar, int lane) {
    const int nb = (R + kBoxRows - 1) / kBoxRows;
    if (lane == 0) mbar_expect_tx(bar, (uint32_t)(2 * nb * kBoxBytes));
    __syncwarp();
    if (lane < 2 * nb) {
        const int half = lane >= nb, i = lane - half * nb;
        tma_box(dst + half * hs + i * kBoxBytes, map, half * 64, row0 + i * kBoxRows, h, b, bar);
    }
}

// The same for the second tensor of a tile longer than SC_TILE_ROWS (V staged where K was): one
// segment [a, e), seeds in seedmask, member masks in the seeds' adjacency rows, counts already known.
__device__ __forceinline__ void merge_long_segment(unsigned char* lane_base, int a, int e, const uint32_t* seedmask,
                                                   const uint32_t* adj, int warp, int lane, int lanes) {
    const int c7 = lane & 7, w_end = (e - 1) >> 5;
    int turn = 0;
    for (int w = a >> 5; w <= w_end; ++w) {
        uint32_t sb = seedmask[w] & bits_between(a, e, w);
        while (sb) {
            const int i = w * 32 + __ffs(sb) - 1;
            sb &= sb - 1;
            if ((turn++ & (kWarps - 1)) != warp) continue;
            const uint32_t* row = adj + adj_row(i) - (i >> 5);
            float sum[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
            int cnt = 0;
            for (int ww = i >> 5; ww <= w_end; ++ww) {
                const uint32_t mem = row[ww];
                cnt += __popc(mem);
                if (lane < lanes) rows_add(lane_base, ww * 32, mem, c7, sum);
            }
            if (cnt > 1 && lane < lanes) row_put_mean(lane_base, i, c7, sum, 1.0f / (float)cnt);
        }
    }
}

template <int kMode, int NL>
__global__ void __launch_bounds__(kThreads, 3) compress_fused_kernel(const __grid_constant__ Params<NL> p) {
    extern __shared__ __align__(1024) unsigned char smem[];   // the swizzle pattern repeats every 1024 bytes
    uint32_t* cnts = reinterpret_cast<uint32_t*>(smem + kCntOff);
    uint32_t* adj = reinterpret_cast<uint32_t*>(smem + kAdjOff);
    float* norm = reinterpret_cast<float*>(smem + kNormOff);
    uint16_t* seedrow = reinterpret_cast<uint16_t*>(smem + kNormOff);   // reuses the norms once they are spent
    int16_t* segs_buf = reinterpret_cast<int16_t*>(smem + kSegsOff);
    uint32_t* seedmask = reinterpret_cast<uint32_t*>(smem + kMiscOff);
    int* geo_buf = reinterpret_cast<int*>(smem + kMiscOff + 32);        // [2][8]
    int* misc = reinterpret_cast<int*>(smem + kMiscOff + 96);           // [0] output offset of the tile, [1] last block,
                                                                        // [2] 32-row blocks that a segment of > 32 tokens touches,
                                                                        // [3] number of segments of more than one token
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + kMiscOff + 272);
    volatile int* umma_failed = reinterpret_cast<volatile int*>(smem + kMiscOff + 276);   // a wait for the tensor core gave up
    int* claim = reinterpret_cast<int*>(smem + kMiscOff + 112);         // next entry of multi[] to be worked on
    uint8_t* multi = smem + kMiscOff + 144;                             // [128] the segments of more than one token
    uint32_t* membits = reinterpret_cast<uint32_t*>(smem + kMiscOff + 288);     // [8] tokens of long segments known to be members
    const uint32_t sbase = smem_u32(smem);
    const uint32_t bar_k = sbase + kBarOff, bar_v = bar_k + 8, bar_u = bar_k + 16;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const bool service = warp == kWarps;   // the ninth warp
    int max_nt = 0;                        // most tiles any sequence has (service warp)

    if (p.skip != nullptr && *p.skip != 0) return;   // uniform over the grid: nothing touched, nothing to clean
    const float tau = p.tau_dev != nullptr ? *p.tau_dev : p.tau;
    // Let the next kernel of the stream start beside this one if it was launched with programmatic stream
    // serialization (a no-op otherwise); this kernel waits for its predecessor only at its very end.
    asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory");
    if (tid == 0) {
        mbar_init(bar_k, 1);
        mbar_init(bar_v, 1);
        mbar_init(bar_u, 1);
        *umma_failed = 0;
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
        if ((sbase & 1023u) != 0u) set_status(p.status, SC_ERR_CUDA);   // the swizzled addressing assumes this
    }
    fence_async_proxy();
    uint32_t phase_k = 0, phase_v = 0, phase_u = 0;
    bool failed = false;
    // Tensor memory for the Gram blocks of long segments: allocated once per (persistent) block by the service warp,
    // which then gives up the permit (a block may not allocate again after that, so it is not done per tile).
    if (warp == kWarps) umma::tmem_alloc(sbase + kMiscOff + 272, kTmemCols);
    umma::fence_before_sync();

    if (service) {
        for (int b = lane; b < p.B; b += 32) max_nt = max(max_nt, min(p.seq_tile_cnt[b], p.n_tile_cap));
        max_nt = warp_max_i(max_nt);
        fetch_tile(p, lane, max_nt, geo_buf, segs_buf);
    }
    if (tid == kNW) { misc[2] = misc[3] = 0; *claim = 0; }
    if (tid >= 32 && tid < 32 + kNW) { seedmask[tid - 32] = 0u; membits[tid - 32] = 0u; }
    __syncthreads();
    umma::fence_after_sync();
    const uint32_t tmem = *tmem_slot;

    int buf = 0;
    for (;;) {
        const int* geo = geo_buf + buf * 8;
        const int16_t* segs = segs_buf + buf * kSegsStride;
        const int t = geo[gT];
        if (t < 0) break;
        const int b = geo[gB], h = geo[gH], nseg = geo[gNseg], row0 = geo[gRow0], R = geo[gR];
        const int bh = b * p.Hkv + h;
        const LayerRefs& lr = p.layer[NL == 1 ? 0 : geo[gLayer]];
        const int unit = (NL == 1 ? 0 : geo[gLayer]) * p.B * p.Hkv + bh;   // index of this (layer, sequence, head)
        const bool long_tile = R > kShortRows;
        const bool two_tensors = (kMode != kCountOnly) && !long_tile;   // V staged beside K
        const int hs = long_tile ? kHalfLong : kHalfShort;

        // ---- 1. stage the rows (service warp, TMA); prefetch ahead ----
        if (service) {
            stage_rows(sbase, hs, &lr.map_k, row0, R, h, b, bar_k, lane);
            if (two_tensors) stage_rows(sbase + kVOff, hs, &lr.map_v, row0, R, h, b, bar_v, lane);
        }
        // end of the segment each row is in (0 past the tile)
        // also: one-token segments (delimiters, lone tokens) are clusters of their own -- no key needed;
        // the others are listed for the warps
        int32_t* as = lr.assign ? lr.assign + (size_t)bh * p.n + row0 : nullptr;
        if (nseg == 1 && R > 1) {
            if (tid == 0) { multi[0] = 0; misc[3] = 1; if (R > kWarpSegMax) misc[2] = (int)((1u << ((R + 31) >> 5)) - 1u); }
        } else {
            for (int s = tid; s < nseg; s += kThreads) {
                const int a = segs[s], e = segs[s + 1];
                if (e - a == 1) {
                    cnts[a] = 1u;
                    atomicOr(&seedmask[a >> 5], 1u << (a & 31));
                    if (as) as[a] = row0 + a;
                    continue;
                }
                multi[atomicAdd(&misc[3], 1)] = (uint8_t)s;
                if (e - a > kWarpSegMax)   // the tile takes the tensor-core step: which 32-row words it concerns
                    for (int k = a >> 5; k <= (e - 1) >> 5; ++k) atomicOr(&misc[2], 1 << k);
            }
        }
        failed = !mbar_wait(bar_k, phase_k);   // K has landed
        phase_k ^= 1u;
        if (two_tensors && !failed) {
            failed = !mbar_wait(bar_v, phase_v);   // and V
            phase_v ^= 1u;
        }
        if (__syncthreads_or(failed)) { failed = true; break; }

        // ---- 2. segments of more than kWarpSegMax tokens: the tile's Gram matrix on the tensor core, 128 x 128 at a
        //         time into tensor memory (one block for a tile of up to 128 tokens, else the two diagonal blocks --
        //         they give the norms -- and the lower one).  Four warps read it, one row per thread, and keep which
        //         earlier tokens of its segment each row is similar to; Algorithm 1 is then settled for all those rows
        //         at once in decision rounds (the sequential pass visits one seed at a time) ----
        if (misc[2] != 0) {
            settle_long_segments(smem, hs, segs, nseg, R, (uint32_t)misc[2], tmem, phase_u, tau, as, row0);
            phase_u ^= 1u;   // one or three blocks
        }

        // ---- 3. the service warp draws the block's next ticket; compute warps: Algorithm 1 for the segments of up
        //         to 32 tokens, one warp each, in registers ----
        unsigned char* lane_base = smem + (lane >> 4) * kVOff + ((lane >> 3) & 1) * hs;   // see rows_add
        if (service) {
            fetch_tile(p, lane, max_nt, geo_buf + (buf ^ 1) * 8, segs_buf + (buf ^ 1) * kSegsStride);
        } else {
            const int nmulti = misc[3];
            for (;;) {   // whichever warp is free takes the next segment
                int k = 0;
                if (lane == 0) k = atomicAdd(claim, 1);
                k = __shfl_sync(kFull, k, 0);
                if (k >= nmulti) break;
                const int s = multi[k];
                const int a = segs[s], e = segs[s + 1];
                if (e - a > kWarpSegMax) continue;   // settled above
                if (tau < 0.f) gsc_short_segment<true>(sbase, hs, a, e - a, tau, norm + warp * 64, seedmask, adj, cnts, as, row0, lane);
                else gsc_short_segment<false>(sbase, hs, a, e - a, tau, norm + warp * 64, seedmask, adj, cnts, as, row0, lane);
            }
        }
        __syncthreads();
        if (*umma_failed) { failed = true; break; }   // a wait for the tensor core gave up in step 2 (known to all by now)

        // ---- 4. cluster count of the tile, published at once.  Service warp: output offset of the tile
        //         (look-back).  Compute warps: the seed row of every cluster, and Eq. 3 ----
        int P = 0;
#pragma unroll
        for (int w = 0; w < kNW; ++w) P += __popc(seedmask[w]);
        uint32_t* stt = p.tile_state + (size_t)unit * p.n_tile_cap;
        if (kMode == kCountOnly) {
            if (tid == 0) {
                if (p.count_into_len) atomicAdd(&lr.core_len[bh], P);
                else stt[t] = (uint32_t)P;
            }
        } else {
            if (!service) {
                if (tid < R) {
                    const uint32_t wbits = seedmask[tid >> 5];
                    if ((wbits >> (tid & 31)) & 1u) {
                        int rank = __popc(wbits & ((1u << (tid & 31)) - 1u));
                        for (int w = 0; w < (tid >> 5); ++w) rank += __popc(seedmask[w]);
                        seedrow[rank] = (uint16_t)tid;
                    }
                }
                compute_warps_sync();   // the table of seed rows is complete
                pool_clusters(lane_base, seedrow, P, adj, cnts, warp, lane, long_tile ? 16 : 32);
            } else {
                if (kMode == kLookBack && lane == 0)
                    atomicExch(&stt[t], (t == 0 ? kFlagPrefix : kFlagAggregate) | (uint32_t)P);
                int base = 0;
                if (kMode == kWriteWithCounts) {
                    for (int k = lane; k < t; k += 32) base += (int)stt[k];
                    base = warp_sum_i(base);
                } else {
                    // look back over the predecessors, nearest first: one poll reads kPollGroups x 32 status
                    // words (the loads overlap), then they are consumed 32 at a time
                    int upto = t;      // tiles [0, upto) still to be accounted for
                    bool gave_up = false, done = false;
                    unsigned long long t0 = 0;
                    while (upto > 0 && !done) {
                        uint32_t v[kPollGroups];
#pragma unroll
                        for (int j = 0; j < kPollGroups; ++j) {
                            const int k = upto - 1 - lane - 32 * j;
                            v[j] = (k >= 0) ? ld_volatile(&stt[k]) : kFlagPrefix;   // before tile 0: prefix 0
                        }
                        bool stalled = false, progressed = false;
#pragma unroll
                        for (int j = 0; j < kPollGroups; ++j) {
                            if (done || stalled) continue;
                            const uint32_t ready = __ballot_sync(kFull, (v[j] >> 30) != 0u);
                            const uint32_t pref = __ballot_sync(kFull, (v[j] >> 30) == 2u);
                            // usable run: lanes 0..m-1 all ready, stopping at the first that holds a full prefix
                            const int first_unready = (ready == kFull) ? 32 : __ffs(~ready) - 1;
                            const int first_pref = pref ? __ffs(pref) - 1 : 32;
                            const int take = min(first_unready, first_pref + 1);
                            const int contrib = (lane < take) ? (int)(v[j] & kValueMask) : 0;
                            base += warp_sum_i(contrib);
                            if (first_pref < first_unready) { done = true; continue; }   // reached an inclusive prefix
                            upto -= take;
                            progressed |= take > 0;
                            stalled = take < 32;
                        }
                        if (!done && !progressed) {
                            if (t0 == 0) t0 = global_ns();
                            else if (global_ns() - t0 > kWaitLimitNs) { gave_up = true; break; }
                            __nanosleep(64);
                        }
                    }
                    if (gave_up) { set_status(p.status, SC_ERR_TIMEOUT); base = 0; }
                    if (lane == 0 && t > 0) atomicExch(&stt[t], kFlagPrefix | (uint32_t)(base + P));
                }
                if (lane == 0) {
                    misc[0] = base;
                    if (geo[gLast]) {
                        lr.core_len[bh] = base + P;
                        if (base + P > p.cap) set_status(p.status, SC_ERR_CAPACITY);
                    }
                }
            }
            __syncthreads();

            // ---- compact, coalesced stores of the cores: cluster `row` of the tile sits in its seed's staged row ----
            const int base = misc[0];
            const size_t obase = (size_t)bh * p.cap;
            for (int idx = tid; idx < P * 16; idx += kThreads) {
                const int row = idx >> 4, c = idx & 15;
                if (base + row < p.cap) {
                    const size_t o = (obase + base + row) * kD + c * 8;
                    const unsigned char* src = smem + (c >> 3) * hs + tile_addr(seedrow[row], c & 7);
                    *reinterpret_cast<uint4*>(lr.core_k + o) = *reinterpret_cast<const uint4*>(src);
                    if (!long_tile) *reinterpret_cast<uint4*>(lr.core_v + o) = *reinterpret_cast<const uint4*>(src + kVOff);
                }
            }
            for (int row = tid; row < P; row += kThreads)
                if (base + row < p.cap)
                    lr.count[obase + base + row] = (int32_t)cnts[seedrow[row]];

            // ---- a tile longer than SC_TILE_ROWS: V takes the place of K and is pooled with the same masks ----
            if (long_tile) {
                fence_async_proxy();   // the copies below overwrite what ordinary accesses read and wrote
                __syncthreads();
                if (service) stage_rows(sbase, hs, &lr.map_v, row0, R, h, b, bar_v, lane);
                failed = !mbar_wait(bar_v, phase_v);
                phase_v ^= 1u;
                if (__syncthreads_or(failed)) { failed = true; break; }
                if (!service) merge_long_segment(lane_base, 0, R, seedmask, adj, warp, lane, 16);
                __syncthreads();
                for (int idx = tid; idx < P * 16; idx += kThreads) {
                    const int row = idx >> 4, c = idx & 15;
                    if (base + row < p.cap)
                        *reinterpret_cast<uint4*>(lr.core_v + (obase + base + row) * kD + c * 8) =
                            *reinterpret_cast<const uint4*>(smem + (c >> 3) * hs + tile_addr(seedrow[row], c & 7));
                }
            }
        }
            if (tid == kNW) { misc[2] = misc[3] = 0; *claim = 0; }
        if (tid >= 32 && tid < 32 + kNW) { seedmask[tid - 32] = 0u; membits[tid - 32] = 0u; }
        fence_async_proxy();   // the next tile's copies overwrite what ordinary accesses read and wrote
        __syncthreads();
        buf ^= 1;
    }

    // ---- exit: the last block to finish leaves the workspace zeroed for the next call ----
    if (failed) {   // a wait gave up: report it, and give copies that may still be in flight one more bounded
                    // wait (either parity: whichever phase is open) before the block's shared memory goes away
        if (tid == 0) set_status(p.status, SC_ERR_TIMEOUT);
        mbar_wait(bar_k, phase_k ^ 1u);
        mbar_wait(bar_v, phase_v ^ 1u);
        mbar_wait(bar_v, phase_v);
    }
    umma::fence_before_sync();
    __syncthreads();
    if (warp == kWarps) umma::tmem_dealloc(tmem, kTmemCols);
    // Under an overlapped launch a block does not finish before the kernel enqueued ahead of this one has
    // completed, so completion is transitive along a run of overlapped launches (a no-op otherwise).
    asm volatile("griddepcontrol.wait;\n" ::: "memory");
    if (tid == 0) {
        __threadfence();
        const int done = atomicAdd(&p.ctl[1], 1);
        misc[1] = (done == (int)gridDim.x - 1);
    }
    __syncthreads();
    if (misc[1]) {
        __threadfence();
        if (kMode != kCountOnly) {
            const size_t words = (size_t)p.L * p.B * p.Hkv * p.n_tile_cap;
            for (size_t i = tid; i < words; i += kThreads) p.tile_state[i] = 0u;
        }
        if (tid == 0) { p.ctl[0] = 0; p.ctl[1] = 0; }
    }
}

}  // namespace cf

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// cuTensorMapEncodeTiled, looked up through the runtime (the library does not link the driver).
EncodeTiledFn encode_tiled() {
    static EncodeTiledFn fn = nullptr;
    if (fn == nullptr) {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
    }
    return fn;
}

// [B, Hkv, n, 128] bf16 with element strides st, read in boxes of 32 rows x 64 columns.
bool make_map(CUtensorMap* map, const void* base, const sc_strides& st, int B, int Hkv, int n) {
    EncodeTiledFn enc = encode_tiled();
    if (enc == nullptr) return false;
    const cuuint64_t dims[4] = {(cuuint64_t)cf::kD, (cuuint64_t)n, (cuuint64_t)Hkv, (cuuint64_t)B};
    const cuuint64_t strides[3] = {(cuuint64_t)st.n * 2, (cuuint64_t)(Hkv > 1 ? st.h : st.n * n) * 2,
                                   (cuuint64_t)(B > 1 ? st.b : st.n * n * (int64_t)Hkv) * 2};
    const cuuint32_t box[4] = {64, (cuuint32_t)cf::kBoxRows, 1, 1};
    const cuuint32_t elem[4] = {1, 1, 1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, elem,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

bool compress_fused_supported(const CompressArgs& a) {
    // ticket arithmetic is 32-bit; TMA strides are below 2^40 bytes
    const int64_t lim = (int64_t)1 << 39;
    return a.dt == SC_BF16 && a.d == cf::kD && a.n_tile_cap >= 1 &&
           (int64_t)a.B * a.Hkv * (int64_t)a.n_tile_cap < (int64_t)1 << 30 && a.st.n > 0 && a.st.n < lim &&
           a.st.h >= 0 && a.st.h < lim && a.st.b >= 0 && a.st.b < lim && encode_tiled() != nullptr;
}

size_t compress_fused_ws_bytes(int32_t B, int32_t Hkv, int32_t n) {
    const size_t tiles = 2 * (size_t)div_up(n, SC_TILE_ROWS) + 1;
    return sizeof(uint32_t) * ((size_t)B * Hkv * tiles + cf::kCtlWords) + 256;
}

namespace {

// Blocks that are resident at once on the current device (one persistent block each), set up on first use.
int resident_blocks() {
    static int grid_of[64] = {0};
    int dev = 0;
    cudaGetDevice(&dev);
    dev &= 63;
    if (grid_of[dev] == 0) {
        cudaFuncSetAttribute(cf::compress_fused_kernel<cf::kCountOnly, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, cf::kSmemBytes);
        cudaFuncSetAttribute(cf::compress_fused_kernel<cf::kWriteWithCounts, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, cf::kSmemBytes);
        cudaFuncSetAttribute(cf::compress_fused_kernel<cf::kLookBack, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, cf::kSmemBytes);
        cudaFuncSetAttribute(cf::compress_fused_kernel<cf::kLookBack, cf::kMaxLayers>, cudaFuncAttributeMaxDynamicSharedMemorySize, cf::kSmemBytes);
        // Blocks per SM by construction: launch bounds (registers), 75 KB of shared memory and 128 of the 512
        // tensor-memory columns each.  (The occupancy query answers 1 for a kernel that allocates tensor memory.)
        // Launching more blocks than are resident would be harmless: a block draws its first ticket when it starts.
        int sms = 0;
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        grid_of[dev] = (sms < 1 ? 1 : sms) * cf::kBlocksPerSm;
    }
    return grid_of[dev];
}

template <int NL>
void fill_common(cf::Params<NL>& p, const CompressArgs& a, int L) {
    p.B = a.B; p.Hkv = a.Hkv; p.n = a.n; p.L = L;
    p.seg_off = a.seg_off; p.tile_seg = a.tile_seg; p.seq_tile_cnt = a.seq_tile_cnt; p.n_tile_cap = a.n_tile_cap;
    p.tau = a.tau; p.cap = a.cap;
    p.tau_dev = a.tau_dev; p.skip = a.skip; p.count_into_len = a.count_only ? 1 : 0;
    p.ctl = (int32_t*)a.ws;
    p.tile_state = (uint32_t*)a.ws + cf::kCtlWords;
    p.status = a.status;
}

bool fill_layer(cf::LayerRefs& r, const CompressArgs& a, const void* K, const void* V, void* core_k, void* core_v,
                int32_t* count, int32_t* core_len, int32_t* assign) {
    r.core_k = (__nv_bfloat16*)core_k; r.core_v = (__nv_bfloat16*)core_v; r.count = count; r.core_len = core_len;
    r.assign = assign;
    return make_map(&r.map_k, K, a.st, a.B, a.Hkv, a.n) && make_map(&r.map_v, V, a.st, a.B, a.Hkv, a.n);
}

}  // namespace

cudaError_t launch_compress_fused(const CompressArgs& a, cudaStream_t st) {
    const int resident = resident_blocks();
    cf::Params<1> p;
    fill_common(p, a, 1);
    if (!fill_layer(p.layer[0], a, a.K, a.V, a.core_k, a.core_v, a.count, a.core_len, a.assign))
        return cudaErrorNotSupported;   // a layout TMA cannot describe: the caller takes the generic kernels
    // no more blocks than there can be tiles
    const int64_t max_tiles = (int64_t)a.B * a.Hkv * a.n_tile_cap;
    const int grid = (int)(max_tiles < resident ? max_tiles : resident);
    if (a.count_only) {   // budget search: per-head cluster counts only
        cf::compress_fused_kernel<cf::kCountOnly, 1><<<grid, cf::kThreads, cf::kSmemBytes, st>>>(p);
        note_launches(1);
    } else if (a.flags & SC_FLAG_TWO_PASS) {
        cf::Params<1> pc = p;
        pc.layer[0].assign = nullptr;
        cf::compress_fused_kernel<cf::kCountOnly, 1><<<grid, cf::kThreads, cf::kSmemBytes, st>>>(pc);
        cf::compress_fused_kernel<cf::kWriteWithCounts, 1><<<grid, cf::kThreads, cf::kSmemBytes, st>>>(p);
        note_launches(2);
    } else {
        // With SC_FLAG_OVERLAP_PREV the kernel may start while the one enqueued before it on the stream is
        // still draining (the caller has promised they share nothing either writes): the tail of one
        // layer's persistent blocks then overlaps the start of the next layer's.
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(grid);
        cfg.blockDim = dim3(cf::kThreads);
        cfg.dynamicSmemBytes = cf::kSmemBytes;
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = (a.flags & SC_FLAG_OVERLAP_PREV) ? 1 : 0;
        note_launches(1);
        return cudaLaunchKernelEx(&cfg, cf::compress_fused_kernel<cf::kLookBack, 1>, p);
    }
    return cudaGetLastError();
}

// Several layers in one launch (sc_compress_layers): the (layer, sequence, head) units take the tickets in turn,
// so consecutive tiles of one head are L*B*Hkv tickets apart and a tile's predecessor has usually published its
// prefix long before the tile looks back.  `a` describes what the layers share (a.K .. a.assign are not used).
cudaError_t launch_compress_fused_layers(const CompressArgs& a, const sc_compress_layer* layers, int32_t L, cudaStream_t st) {
    if (L < 1 || L > cf::kMaxLayers) return cudaErrorInvalidValue;
    const int resident = resident_blocks();
    static cf::Params<cf::kMaxLayers> p;   // 20 KB: kept off the stack; filled and passed by value under the lock
    static std::mutex lock;
    std::lock_guard<std::mutex> guard(lock);
    fill_common(p, a, L);
    for (int l = 0; l < L; ++l)
        if (!fill_layer(p.layer[l], a, layers[l].K, layers[l].V, layers[l].core_k, layers[l].core_v, layers[l].count,
                        layers[l].core_len, layers[l].assign))
            return cudaErrorNotSupported;
    for (int l = L; l < cf::kMaxLayers; ++l) p.layer[l] = p.layer[0];
    const int64_t max_tiles = (int64_t)L * a.B * a.Hkv * a.n_tile_cap;
    const int grid = (int)(max_tiles < resident ? max_tiles : resident);
    cf::compress_fused_kernel<cf::kLookBack, cf::kMaxLayers><<<grid, cf::kThreads, cf::kSmemBytes, st>>>(p);
    note_launches(1);
    return cudaGetLastError();
}

size_t compress_fused_layers_ws_bytes(int32_t L, int32_t B, int32_t Hkv, int32_t n) {
    const size_t tiles = 2 * (size_t)div_up(n, SC_TILE_ROWS) + 1;
    return sizeof(uint32_t) * ((size_t)L * B * Hkv * tiles + cf::kCtlWords) + 256;
}

}  // namespace sc

