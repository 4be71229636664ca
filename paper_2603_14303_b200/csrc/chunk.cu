// sc_chunk: delimiter-bounded chunking (Sec. 2.2, Eq. 1) as a segmented boundary scan.
//
// Per sequence position p: isd[p] = token id in the delimiter set.  A non-delimiter run starts
// at p when p == 0 or isd[p-1]; run_start(p) is the running maximum of those positions, and p
// opens a segment iff isd[p] or (p - run_start(p)) % max_chunk_len == 0.  Segment offsets are
// the compacted positions of those flags.  Four small kernels over 2048-token tiles (no
// inter-block waiting), then one block per sequence packs consecutive segments into the
// <= SC_TILE_ROWS-token work tiles sc_compress consumes.
#include "common.cuh"

namespace sc {

constexpr int kChunkThreads = 256;
constexpr int kChunkPer = 8;
constexpr int kChunkTile = kChunkThreads * kChunkPer;  // 2048 tokens per block
constexpr int kPackWindow = 4096;

struct DelimSet {
    int32_t id[SC_MAX_DELIMS];
    int32_t n;
};

__device__ __forceinline__ bool in_set(int32_t tok, const DelimSet& D) {
    bool hit = false;
    for (int i = 0; i < D.n; ++i) hit |= (D.id[i] == tok);
    return hit;
}

// Block-wide inclusive scan of one int per thread (sum or max), 256 threads.
template <bool kMax>
__device__ __forceinline__ int block_scan(int v, int* warp_tot /*[8]*/, int* block_total) {
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    int s = kMax ? warp_scan_max(v, lane) : warp_scan_add(v, lane);
    if (lane == 31) warp_tot[w] = s;
    __syncthreads();
    int carry = kMax ? -1 : 0, tot = kMax ? -1 : 0;
    for (int i = 0; i < kChunkThreads / 32; ++i) {
        int t = warp_tot[i];
        if (i < w) carry = kMax ? max(carry, t) : carry + t;
        tot = kMax ? max(tot, t) : tot + t;
    }
    __syncthreads();
    *block_total = tot;
    return kMax ? max(s, carry) : s + carry;
}

// Loads this thread's 8 consecutive tokens and the one before them; returns delimiter bits
// (bit i = token i is a delimiter, bit 8 = the token before is one / sequence start marker).
__device__ __forceinline__ void load_flags(const int32_t* ids, int n, int p0, const DelimSet& D,
                                           unsigned& isd_bits, bool& prev_isd) {
    isd_bits = 0;
#pragma unroll
    for (int i = 0; i < kChunkPer; ++i) {
        int p = p0 + i;
        if (p < n && in_set(ids[p], D)) isd_bits |= 1u << i;
    }
    prev_isd = (p0 > 0 && p0 - 1 < n) ? in_set(ids[p0 - 1], D) : false;
}

// Kernel 1: last run-start position inside each tile (-1 if none).
__global__ void __launch_bounds__(kChunkThreads)
chunk_tile_last(const int32_t* __restrict__ token_ids, int n, int tps, DelimSet D, int32_t* __restrict__ tile_last) {
    const int b = blockIdx.x / tps, tile = blockIdx.x % tps;
    const int32_t* ids = token_ids + (int64_t)b * n;
    const int p0 = tile * kChunkTile + threadIdx.x * kChunkPer;
    unsigned isd; bool prev;
    load_flags(ids, n, p0, D, isd, prev);
    int last = -1;
#pragma unroll
    for (int i = 0; i < kChunkPer; ++i) {
        int p = p0 + i;
        bool pv = (i == 0) ? prev : ((isd >> (i - 1)) & 1u);
        if (p < n && (p == 0 || pv)) last = p;
    }
    __shared__ int wt[kChunkThreads / 32];
    int tot;
    block_scan<true>(last, wt, &tot);
    if (threadIdx.x == 0) tile_last[blockIdx.x] = tot;
}

// Segment-start flags of this thread's 8 tokens, given the run start carried into the tile.
__device__ __forceinline__ unsigned start_flags(int n, int p0, unsigned isd, bool prev, int carry_in,
                                                int max_len, int* wt) {
    // thread-local inclusive max of run-start candidates, then block scan of the thread maxima
    int cand[kChunkPer];
    int tmax = -1;
#pragma unroll
    for (int i = 0; i < kChunkPer; ++i) {
        int p = p0 + i;
        bool pv = (i == 0) ? prev : ((isd >> (i - 1)) & 1u);
        cand[i] = (p < n && (p == 0 || pv)) ? p : -1;
        tmax = max(tmax, cand[i]);
    }
    int tot;
    int incl = block_scan<true>(tmax, wt, &tot);
    // exclusive value for this thread = max over earlier threads and the carry
    int excl = __shfl_up_sync(kFull, incl, 1);
    if ((threadIdx.x & 31) == 0) excl = -1;
    __shared__ int warp_excl[kChunkThreads / 32];
    if ((threadIdx.x & 31) == 31) warp_excl[threadIdx.x >> 5] = incl;
    __syncthreads();
    if ((threadIdx.x & 31) == 0 && threadIdx.x > 0) excl = warp_excl[(threadIdx.x >> 5) - 1];
    __syncthreads();
    int run = max(excl, carry_in);
    unsigned flags = 0;
#pragma unroll
    for (int i = 0; i < kChunkPer; ++i) {
        int p = p0 + i;
        run = max(run, cand[i]);
        if (p < n) {
            bool d = (isd >> i) & 1u;
            if (d || ((p - run) % max_len) == 0) flags |= 1u << i;
        }
    }
    return flags;
}

__device__ __forceinline__ int carry_into_tile(const int32_t* tile_last, int b, int tps, int tile) {
    // run start carried in from the earlier tiles of the same sequence (tps is small: n / 2048)
    int c = -1;
    for (int t = threadIdx.x; t < tile; t += kChunkThreads) c = max(c, tile_last[b * tps + t]);
    __shared__ int wt2[kChunkThreads / 32];
    c = warp_max_i(c);
    if ((threadIdx.x & 31) == 0) wt2[threadIdx.x >> 5] = c;
    __syncthreads();
    int r = -1;
    for (int i = 0; i < kChunkThreads / 32; ++i) r = max(r, wt2[i]);
    __syncthreads();
    return r;
}

// Kernel 2: number of segment starts per tile.
__global__ void __launch_bounds__(kChunkThreads)
chunk_tile_count(const int32_t* __restrict__ token_ids, int n, int tps, DelimSet D, int max_len,
                 const int32_t* __restrict__ tile_last, int32_t* __restrict__ tile_cnt) {
    const int b = blockIdx.x / tps, tile = blockIdx.x % tps;
    const int32_t* ids = token_ids + (int64_t)b * n;
    const int p0 = tile * kChunkTile + threadIdx.x * kChunkPer;
    __shared__ int wt[kChunkThreads / 32];
    unsigned isd; bool prev;
    load_flags(ids, n, p0, D, isd, prev);
    int carry = carry_into_tile(tile_last, b, tps, tile);
    unsigned flags = start_flags(n, p0, isd, prev, carry, max_len, wt);
    int tot;
    block_scan<false>(__popc(flags), wt, &tot);
    if (threadIdx.x == 0) tile_cnt[blockIdx.x] = tot;
}

// Kernel 3: one block scans the tile counts -> tile bases, n_seg, seq_seg_off.
__global__ void __launch_bounds__(kChunkThreads)
chunk_scan_tiles(int B, int n, int tps, const int32_t* __restrict__ tile_cnt, int32_t* __restrict__ tile_base,
                 int32_t* __restrict__ seq_seg_off, int32_t* __restrict__ n_seg, int32_t* __restrict__ seg_off,
                 int n_seg_cap, int32_t* status) {
    __shared__ int wt[kChunkThreads / 32];
    const int total_tiles = B * tps;
    int carry = 0;
    for (int base = 0; base < total_tiles; base += kChunkThreads) {
        int i = base + threadIdx.x;
        int v = (i < total_tiles) ? tile_cnt[i] : 0;
        int tot;
        int incl = block_scan<false>(v, wt, &tot);
        if (i < total_tiles) {
            int excl = carry + incl - v;
            tile_base[i] = excl;
            if (i % tps == 0) seq_seg_off[i / tps] = excl;
        }
        carry += tot;
    }
    if (threadIdx.x == 0) {
        seq_seg_off[B] = carry;
        *n_seg = carry;
        if (carry > n_seg_cap) set_status(status, SC_ERR_CAPACITY);
        else seg_off[carry] = B * n;
    }
}

// Kernel 4: write the compacted segment offsets.
__global__ void __launch_bounds__(kChunkThreads)
chunk_write(const int32_t* __restrict__ token_ids, int n, int tps, DelimSet D, int max_len,
            const int32_t* __restrict__ tile_last, const int32_t* __restrict__ tile_base,
            int32_t* __restrict__ seg_off, int n_seg_cap) {
    const int b = blockIdx.x / tps, tile = blockIdx.x % tps;
    const int32_t* ids = token_ids + (int64_t)b * n;
    const int p0 = tile * kChunkTile + threadIdx.x * kChunkPer;
    __shared__ int wt[kChunkThreads / 32];
    unsigned isd; bool prev;
    load_flags(ids, n, p0, D, isd, prev);
    int carry = carry_into_tile(tile_last, b, tps, tile);
    unsigned flags = start_flags(n, p0, isd, prev, carry, max_len, wt);
    int cnt = __popc(flags), tot;
    int incl = block_scan<false>(cnt, wt, &tot);
    int rank = tile_base[blockIdx.x] + incl - cnt;
#pragma unroll
    for (int i = 0; i < kChunkPer; ++i) {
        if ((flags >> i) & 1u) {
            if (rank < n_seg_cap) seg_off[rank] = b * n + p0 + i;
            ++rank;
        }
    }
}

// Kernel 5: one block per sequence packs consecutive segments into work tiles: as many whole
// segments as fit in SC_TILE_ROWS tokens, or one longer segment alone.  The chain tile -> next tile is
// sequential, but where a tile that starts at segment s ends does not depend on the chain: the
// sequence's offsets are staged through shared memory in windows, every thread finds the end of the
// tile that would start at its segments (a binary search over the monotone offsets), and one thread then
// walks the chain with a single shared-memory lookup per tile.
__global__ void __launch_bounds__(kChunkThreads)
chunk_pack_tiles(const int32_t* __restrict__ seg_off, const int32_t* __restrict__ seq_seg_off, int n_seg_cap,
                 int32_t* __restrict__ tile_seg, int n_tile_cap, int32_t* __restrict__ seq_tile_cnt,
                 int32_t* status) {
    __shared__ int buf[kPackWindow + 1];
    __shared__ int nxt[kPackWindow];       // window index of the segment the next tile starts at
    __shared__ int sh_cur, sh_nt;
    const int b = blockIdx.x;
    const int s0 = seq_seg_off[b];
    const int s1 = min(seq_seg_off[b + 1], n_seg_cap);  // clamped when sc_chunk overflowed
    int32_t* out = tile_seg + (int64_t)b * (n_tile_cap + 1);
    int cur = s0, nt = 0;
    while (cur < s1) {
        const int ws = cur;
        const int cnt = min(kPackWindow, s1 - ws);
        for (int i = threadIdx.x; i <= cnt; i += kChunkThreads) buf[i] = seg_off[ws + i];
        __syncthreads();
        for (int i = threadIdx.x; i < cnt; i += kChunkThreads) {
            // largest e in (i, cnt] with buf[e] - buf[i] <= SC_TILE_ROWS, or i + 1 for a segment longer than a tile
            const int limit = buf[i] + SC_TILE_ROWS;
            int lo = i + 1, hi = min(cnt, i + SC_TILE_ROWS);   // a segment holds at least one token
            while (lo < hi) {
                const int mid = (lo + hi + 1) >> 1;
                if (buf[mid] <= limit) lo = mid; else hi = mid - 1;
            }
            nxt[i] = lo;
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            // a tile's end is known for sure only if SC_TILE_ROWS + 1 offsets behind its start are in the window
            const bool last_window = (ws + cnt == s1);
            while (cur < s1 && (last_window || cur - ws + SC_TILE_ROWS + 1 <= cnt)) {
                if (nt < n_tile_cap) out[nt] = cur;
                ++nt;
                cur = ws + nxt[cur - ws];
            }
            sh_cur = cur; sh_nt = nt;
        }
        __syncthreads();
        cur = sh_cur; nt = sh_nt;
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        out[min(nt, n_tile_cap)] = s1;
        seq_tile_cnt[b] = nt;
        if (nt > n_tile_cap) set_status(status, SC_ERR_CAPACITY);
    }
}

size_t chunk_ws_bytes(int32_t B, int32_t n) {
    int tps = div_up(n, kChunkTile);
    return sizeof(int32_t) * 3 * (size_t)B * tps + 64;
}

cudaError_t launch_chunk(const ChunkArgs& a, cudaStream_t st) {
    const int tps = div_up(a.n, kChunkTile);
    const int tiles = a.B * tps;
    int32_t* tile_last = a.ws;
    int32_t* tile_cnt = a.ws + tiles;
    int32_t* tile_base = a.ws + 2 * tiles;
    DelimSet D;
    D.n = a.n_delim;
    for (int i = 0; i < SC_MAX_DELIMS; ++i) D.id[i] = (i < a.n_delim) ? a.delim[i] : 0;
    chunk_tile_last<<<tiles, kChunkThreads, 0, st>>>(a.token_ids, a.n, tps, D, tile_last);
    chunk_tile_count<<<tiles, kChunkThreads, 0, st>>>(a.token_ids, a.n, tps, D, a.max_chunk_len, tile_last, tile_cnt);
    chunk_scan_tiles<<<1, kChunkThreads, 0, st>>>(a.B, a.n, tps, tile_cnt, tile_base, a.seq_seg_off, a.n_seg,
                                                  a.seg_off, a.n_seg_cap, a.status);
    chunk_write<<<tiles, kChunkThreads, 0, st>>>(a.token_ids, a.n, tps, D, a.max_chunk_len, tile_last, tile_base,
                                                 a.seg_off, a.n_seg_cap);
    chunk_pack_tiles<<<a.B, kChunkThreads, 0, st>>>(a.seg_off, a.seq_seg_off, a.n_seg_cap, a.tile_seg,
                                                    a.n_tile_cap, a.seq_tile_cnt, a.status);
    note_launches(5);
    return cudaGetLastError();
}

}  // namespace sc
