/*
 * SemantiCache hot path for NVIDIA B200 (sm_100a) -- C ABI.
 *
 * Three calls follow the paper's pipeline:
 *   sc_chunk        Sec. 2.2, Eq. 1          token ids + delimiter set -> chunk offsets
 *   sc_compress     Sec. 2.3-2.4, Eq. 2,     per layer: K/V + chunk offsets + GSC parameters ->
 *                   Algorithm 1, Eq. 3       semantic cores (K, V), member counts, per-head lengths
 *   sc_decode_attn  Sec. 2.4, Eq. 4          GQA decode queries against the cores with
 *                                            Proportional Attention (softmax(qK^T/sqrt(d) + ln s) V)
 *
 * General rules
 *   - Every pointer is a DEVICE pointer unless its comment says HOST.  The caller owns all
 *     buffers; the library allocates nothing.  The state it keeps between calls: the launch
 *     counter, per-GPU launch geometry looked up on first use, and, for sc_decode_attn_static
 *     only, its fixed scratch array with the per-GPU address of that array.
 *   - All work is enqueued on `stream` (a cudaStream_t passed as void*; NULL = default stream).
 *     Calls return after enqueueing; they never synchronise.
 *   - The return value reports host-side validation only (SC_OK, SC_ERR_INVALID_ARG,
 *     SC_ERR_UNSUPPORTED, SC_ERR_CUDA for a failed launch; sc_decode_attn_static alone also
 *     returns SC_ERR_CAPACITY from the host for a shape beyond its fixed scratch).  Conditions found on the device
 *     are written to the caller's `status` word (int32, device or pinned host memory, may be
 *     NULL): it is left untouched on success and set to SC_ERR_CAPACITY / SC_ERR_TIMEOUT
 *     otherwise (first error wins).  The caller zeroes it beforehand.  Kernels never trap.
 *   - Tensors are row-major with the head dimension d innermost and contiguous; device
 *     pointers of K, V, q, cores and out must be 16-byte aligned.  d must be 128 for SC_BF16
 *     fast paths; the generic path takes any d that is a multiple of 8 up to 256.
 *   - Results are deterministic: the same inputs give bit-identical outputs.
 */
#ifndef SEMANTICACHE_H_
#define SEMANTICACHE_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define SC_API __attribute__((visibility("default")))
#else
#define SC_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    SC_OK = 0,
    SC_ERR_INVALID_ARG = 1,
    SC_ERR_UNSUPPORTED = 2,
    SC_ERR_CAPACITY = 3,
    SC_ERR_CUDA = 4,
    SC_ERR_TIMEOUT = 5
} sc_status;

typedef enum { SC_BF16 = 0, SC_F32 = 1 } sc_dtype;

/* sc_gsc_params.flags */
#define SC_FLAG_GENERIC 1u     /* force the generic (CUDA-core, any dtype) kernels */
#define SC_FLAG_TWO_PASS 2u    /* fused compress: count pass + write pass instead of the
                                  single pass whose tiles look back for their output offset */
#define SC_FLAG_OVERLAP_PREV 4u /* sc_decode_attn, sc_compress (fused bf16 path, single pass): launch with
                                  programmatic stream serialization, so that this kernel may start while
                                  the kernels enqueued before it on this stream are still running.  The
                                  caller promises that nothing this call READS before it writes (q, cores,
                                  count, core_len; for sc_compress K, V and the chunk plan) is written by
                                  any kernel of the unbroken run of overlapped launches before it, nor by
                                  the kernel just before that run.  Every write of the call (out,
                                  workspace, status; for sc_compress also cores, count, core_len, assign)
                                  is ordered behind the completion of the kernel before it, and so on
                                  back along the run: sc_decode_attn calls of one run may therefore share
                                  their workspace and out buffers; sc_compress calls of one run must not
                                  share a workspace or outputs (it writes throughout).  Independent
                                  calls, e.g. the layers of an attention-only benchmark, then run back to
                                  back without the launch gap.  A call without the flag orders itself
                                  after everything enqueued before it, as usual. */
#define SC_FLAG_OVERLAP_CHAIN 8u /* sc_decode_attn only: as SC_FLAG_OVERLAP_PREV, except that q MAY be the
                                  product of the kernel just before this call (layer l+1's query follows
                                  from layer l's output).  The kernel starts early, sends its share of the
                                  cores on its way (first tiles to shared memory, the rest to L2), waits
                                  for the preceding kernel to complete and only then reads q.  The cores,
                                  count and core_len are still read early and fall under the promise
                                  above.  Ignored (ordinary launch) on the generic path. */

#define SC_FLAG_CAUSAL_TAIL 16u /* sc_prefill_attn only: the last m rows of every head are the m queries' own
                                  tokens; query i attends to rows t < core_len - (m - 1 - i) */

typedef struct {
    float tau;             /* similarity threshold of Algorithm 1; merge iff Sim > tau (strict) */
    int32_t max_chunk_len; /* must equal the value given to sc_chunk; 1..SC_MAX_CHUNK_LEN */
    uint32_t flags;        /* SC_FLAG_* */
} sc_gsc_params;

/* Element strides of a [B, Hkv, n, d] tensor (d contiguous). */
typedef struct { int64_t b, h, n; } sc_strides;

#define SC_MAX_CHUNK_LEN 256
#define SC_MAX_DELIMS 64
#define SC_TILE_ROWS 128       /* rows a compress tile packs (one longer chunk is a tile alone) */

/* Library / build identification: returns a static string. */
SC_API const char* sc_version(void);

/*
 * Statistics: number of kernels this library has launched (or recorded into a CUDA graph under
 * stream capture) since it was loaded.  It affects nothing.
 */
SC_API uint64_t sc_launch_counter(void);

/*
 * Upper bounds for the outputs of sc_chunk, so a caller can allocate without a sync:
 * segments <= *n_seg_cap = B*n in total, tiles <= *n_tile_cap per sequence.  Both pointers are HOST.
 */
SC_API sc_status sc_chunk_bounds(int32_t B, int32_t n, int32_t* n_seg_cap /*HOST out*/,
                          int32_t* n_tile_cap /*HOST out*/);

/*
 * Semantic chunking (Sec. 2.2, Eq. 1).  The token axis of each sequence is cut into the
 * alternating series (C_1, d_1, C_2, ...): every maximal run of non-delimiter tokens is one
 * segment, cut every max_chunk_len tokens if longer; every delimiter token is a segment of
 * length one (clustering a one-token segment returns the token unchanged, which is how the
 * delimiters' K/V stay unmodified); empty runs produce nothing; no segment spans sequences.
 * Depends on token ids only, so one call serves every layer and KV head.
 *
 *   token_ids    [B, n] int32
 *   delim_ids    HOST, n_delim <= SC_MAX_DELIMS ids
 *   seg_off      out [n_seg+1]: start of each segment on the flattened [B*n] axis, then B*n.
 *                Capacity n_seg_cap+1 entries.
 *   seq_seg_off  out [B+1]: first segment of each sequence, then n_seg
 *   n_seg        out [1]
 *   tile_seg     out [B, n_tile_cap+1]: work partition for sc_compress.  Row b lists the tiles of
 *                sequence b: tile t covers segments [tile_seg[b][t], tile_seg[b][t+1]) -- as many
 *                consecutive segments as fit in SC_TILE_ROWS tokens, or one longer segment
 *                alone.  n_tile_cap from sc_chunk_bounds always suffices.
 *   seq_tile_cnt out [B]: number of tiles of each sequence
 *   workspace    scratch of at least sc_chunk_workspace_bytes(B, n) bytes
 *   status       SC_ERR_CAPACITY if n_seg > n_seg_cap or a sequence needs more than n_tile_cap
 *                tiles (writes clamped; n_seg and seq_tile_cnt still report the needed sizes)
 * B == 0 or n == 0 is valid and yields empty offsets.
 */
SC_API size_t sc_chunk_workspace_bytes(int32_t B, int32_t n);

SC_API sc_status sc_chunk(const int32_t* token_ids, int32_t B, int32_t n,
                   const int32_t* delim_ids /*HOST*/, int32_t n_delim, int32_t max_chunk_len,
                   int32_t* seg_off, int32_t n_seg_cap, int32_t* seq_seg_off, int32_t* n_seg,
                   int32_t* tile_seg, int32_t n_tile_cap, int32_t* seq_tile_cnt,
                   void* workspace, size_t workspace_bytes, int32_t* status, void* stream);

/*
 * Compress one layer (Sec. 2.3-2.4).  For every (sequence b, KV head h, segment) independently:
 * Greedy Seed-Based Clustering (Algorithm 1) on the cosine similarity of the keys (Eq. 2; a
 * zero-norm key has similarity 0 to everything), then each cluster S_t is mean-pooled into one
 * core k_hat = mean(k_i), v_hat = mean(v_i) (Eq. 3; fp32 accumulation, rounded once to
 * the storage dtype) with count = |S_t|.  Cores are written compactly in position order of
 * their seeds; a delimiter is a core of count 1 carrying its K/V bits unchanged.
 *
 *   K, V        [B, Hkv, n, d] with element strides kv_strides (both tensors), dtype dt
 *   seg_off .. seq_tile_cnt, n_tile_cap   as produced by / given to sc_chunk for the same B, n,
 *               max_chunk_len
 *   params      HOST
 *   core_k/v    out [B, Hkv, cap, d] contiguous, dtype dt; rows < core_len[b,h] are valid
 *   count       out [B, Hkv, cap] int32, >= 1 on valid rows
 *   core_len    out [B, Hkv]: number of cores of each head (the needed length even when it
 *               exceeds cap; then status = SC_ERR_CAPACITY and rows >= cap are not written).
 *               cap = n always suffices.
 *   assign      optional out [B, Hkv, n] int32: for each token the position (within its
 *               sequence) of the seed of its cluster; NULL to skip
 *   workspace   at least sc_compress_workspace_bytes(B, Hkv, n) bytes.  It holds per-tile status
 *               words and two counters that must be zero on entry and are left zero on exit, so
 *               zero the workspace once after allocating it (and again after a call that
 *               reported SC_ERR_TIMEOUT).  Calls that share a workspace must not overlap.
 */
SC_API size_t sc_compress_workspace_bytes(int32_t B, int32_t Hkv, int32_t n);

SC_API sc_status sc_compress(const void* K, const void* V, sc_strides kv_strides, sc_dtype dt,
                      int32_t B, int32_t Hkv, int32_t n, int32_t d,
                      const int32_t* seg_off, const int32_t* seq_seg_off, const int32_t* n_seg,
                      const int32_t* tile_seg, const int32_t* seq_tile_cnt, int32_t n_tile_cap,
                      const sc_gsc_params* params /*HOST*/,
                      void* core_k, void* core_v, int32_t* count, int32_t cap, int32_t* core_len,
                      int32_t* assign, void* workspace, size_t workspace_bytes,
                      int32_t* status, void* stream);

/*
 * sc_compress for several layers of a model in one launch (same results, layer by layer).  At the end of
 * a prefill every layer's K and V exist, and all layers share the chunk plan (it depends on token ids
 * only): one call then replaces L, and the kernel has L times as many independent (layer, sequence, head)
 * units to interleave, which matters when a layer alone has few of them.
 *
 *   layers      HOST array of L rows of DEVICE pointers: K, V (both with kv_strides), core_k, core_v,
 *               count, core_len, assign (or NULL) as sc_compress takes them for that layer.  Layers must
 *               not share outputs.  The array is read during the call only.
 *   L           1..SC_MAX_LAYERS_PER_CALL
 *   the rest    as for sc_compress; params->flags may hold SC_FLAG_GENERIC only (the generic kernels then
 *               run layer after layer)
 *   workspace   at least sc_compress_layers_workspace_bytes(L, B, Hkv, n) bytes, zeroed once after
 *               allocation and left zeroed by every call
 */
typedef struct {
    const void* K; const void* V;
    void* core_k; void* core_v; int32_t* count; int32_t* core_len; int32_t* assign;
} sc_compress_layer;

#define SC_MAX_LAYERS_PER_CALL 64

SC_API size_t sc_compress_layers_workspace_bytes(int32_t L, int32_t B, int32_t Hkv, int32_t n);

SC_API sc_status sc_compress_layers(const sc_compress_layer* layers /*HOST [L]*/, int32_t L, sc_strides kv_strides,
                             sc_dtype dt, int32_t B, int32_t Hkv, int32_t n, int32_t d,
                             const int32_t* seg_off, const int32_t* seq_seg_off, const int32_t* n_seg,
                             const int32_t* tile_seg, const int32_t* seq_tile_cnt, int32_t n_tile_cap,
                             const sc_gsc_params* params /*HOST*/, int32_t cap,
                             void* workspace, size_t workspace_bytes, int32_t* status, void* stream);

/*
 * Compress one layer to a KV budget (the paper evaluates budgets of 20 / 35 / 50 % kept, Table 1, and
 * shows that a lower threshold keeps fewer entries, Table 4b; how a budget is turned into a threshold
 * it does not say).  This library's reading: the threshold of Algorithm 1 is searched on a grid
 *     tau_i = tau_lo + i * ((tau_hi - tau_lo) / (n_grid - 1)),  i = 0 .. n_grid - 1   (float32 arithmetic)
 * for the value whose number of cores, all sequences and KV heads of the layer together, comes
 * nearest to target = floor(target_kept * B * Hkv * n + 0.5), assuming that the count does not fall
 * as the threshold rises:
 *   1. the lowest threshold is counted; if it already keeps at least the target it is chosen;
 *      else the highest is counted; if even that keeps less than the target it is chosen;
 *   2. otherwise the interval is halved (middle index, rounded down) until its ends are adjacent,
 *      with "fewer than the target" at the lower end and "at least the target" at the upper;
 *   3. of the two ends the one whose count is nearer the target is chosen, the lower on a tie.
 * Everything runs on the device without a host round trip: at most 2 + ceil(log2(n_grid - 1))
 * counting passes (Eq. 2 + Algorithm 1 on the keys alone, no Eq. 3, nothing written but counts),
 * each followed by a one-block step that moves the search on, then one ordinary compress pass at
 * the chosen threshold.  Counting passes enqueued after the choice is made return at once.
 *
 *   K .. n_tile_cap, core_k .. assign, status   as for sc_compress; params->tau is ignored;
 *               params->flags may hold SC_FLAG_GENERIC only.  B, n > 0.
 *   budget      HOST: target_kept in [0, 1], tau_lo < tau_hi, n_grid in [2, SC_BUDGET_MAX_GRID]
 *   tau_out     out [1] float (device), may be NULL: the chosen threshold
 *   search_out  out [2] int32 (device), may be NULL: the chosen grid index, and the number of
 *               counting passes that did work
 *   workspace   at least sc_compress_budget_workspace_bytes(B, Hkv, n) bytes, zeroed once after
 *               allocation like sc_compress's (and left ready for the next call)
 */
typedef struct {
    float target_kept;     /* wanted cores / tokens of the layer */
    float tau_lo, tau_hi;  /* ends of the threshold grid */
    int32_t n_grid;        /* number of grid points */
} sc_budget;

#define SC_BUDGET_MAX_GRID 65

SC_API size_t sc_compress_budget_workspace_bytes(int32_t B, int32_t Hkv, int32_t n);

SC_API sc_status sc_compress_budget(const void* K, const void* V, sc_strides kv_strides, sc_dtype dt,
                             int32_t B, int32_t Hkv, int32_t n, int32_t d,
                             const int32_t* seg_off, const int32_t* seq_seg_off, const int32_t* n_seg,
                             const int32_t* tile_seg, const int32_t* seq_tile_cnt, int32_t n_tile_cap,
                             const sc_gsc_params* params /*HOST*/, const sc_budget* budget /*HOST*/,
                             void* core_k, void* core_v, int32_t* count, int32_t cap, int32_t* core_len,
                             int32_t* assign, float* tau_out, int32_t* search_out,
                             void* workspace, size_t workspace_bytes, int32_t* status, void* stream);

/*
 * Compress one layer WITHOUT chunking: the "none / global" arm of the paper's chunking ablation
 * (Table 4a).  Algorithm 1 (Sec. 2.3) runs over each whole sequence as a single chunk -- delimiters
 * get no special treatment, a token may join a seed anywhere before it -- and every cluster is then
 * mean-pooled by Eq. 3 (Sec. 2.4) exactly as in sc_compress: cores in position order of their seeds,
 * count = |S_t|, fp32 sums in token order, one rounding.
 *
 * Algorithm 1 over n tokens is evaluated through its closed form (the seeds are the first maximal
 * independent set, in index order, of the graph Sim > tau; every other token joins its lowest adjacent
 * seed): all pairwise similarities of a head are thresholded into a bit matrix (tensor cores for
 * SC_BF16 with d = 128, CUDA cores otherwise), then seeds and members are decided in parallel rounds.
 * The result is the one a sequential run gives.  Cost grows with n^2: about n^2 / 16 bytes of
 * workspace per (sequence, head) and n^2 * d multiply-adds.
 *
 *   K, V, kv_strides, dt, core_k .. assign, status   as for sc_compress (assign: position of each token's seed)
 *   n          at most SC_GLOBAL_MAX_TOKENS;  B * Hkv at most 65535
 *   flags      SC_FLAG_GENERIC forces the CUDA-core similarity kernel; else 0
 *   workspace  at least sc_compress_global_workspace_bytes(B, Hkv, n) bytes, 16-byte aligned; no
 *              initialisation needed, nothing persists between calls
 */
#define SC_GLOBAL_MAX_TOKENS 131072

SC_API size_t sc_compress_global_workspace_bytes(int32_t B, int32_t Hkv, int32_t n);

SC_API sc_status sc_compress_global(const void* K, const void* V, sc_strides kv_strides, sc_dtype dt,
                             int32_t B, int32_t Hkv, int32_t n, int32_t d, float tau, uint32_t flags,
                             void* core_k, void* core_v, int32_t* count, int32_t cap, int32_t* core_len,
                             int32_t* assign, void* workspace, size_t workspace_bytes, int32_t* status, void* stream);

/*
 * One decode step of Proportional Attention (Sec. 2.4, Eq. 4) for one layer.  For every query
 * head hq of sequence b, with KV head h = hq / (Hq/Hkv):
 *     x_t = scale * <q, k_hat_t> + ln(count_t),  out = sum_t softmax(x)_t * v_hat_t
 * over rows t < core_len[b, h].  The whole query group of a KV head is served in one pass over
 * that head's cores; long heads are split along t and the partial (max, sum, acc) triples are
 * combined by the last block to finish.
 *
 *   q          [B, Hq, d] contiguous, dtype dt
 *   core_k/v   [B, Hkv, cap, d] contiguous, dtype dt;  count [B, Hkv, cap] int32, or NULL for
 *              all ones (plain attention over an uncompressed cache)
 *   core_len   [B, Hkv] int32 (device), each <= cap
 *   scale      0 means 1/sqrt(d)
 *   out        [B, Hq, d] contiguous, dtype dt; a head with core_len 0 gets zeros
 *   flags      SC_FLAG_GENERIC forces the generic kernels; SC_FLAG_OVERLAP_PREV or
 *              SC_FLAG_OVERLAP_CHAIN (see above); else 0
 *   workspace  at least sc_decode_workspace_bytes(B, Hq, Hkv, d, cap) bytes.  It holds the
 *              split partials and a few arrival counters; the counters must be zero on entry
 *              and are left zero on exit, so zero the workspace once after allocating it.
 */
SC_API size_t sc_decode_workspace_bytes(int32_t B, int32_t Hq, int32_t Hkv, int32_t d, int32_t cap);

SC_API sc_status sc_decode_attn(const void* q, sc_dtype dt, int32_t B, int32_t Hq, int32_t Hkv, int32_t d,
                         const void* core_k, const void* core_v, const int32_t* count, int32_t cap,
                         const int32_t* core_len, float scale, uint32_t flags, void* out,
                         void* workspace, size_t workspace_bytes, int32_t* status, void* stream);

/*
 * Proportional Attention for a block of m queries per head (Sec. 2.4, Eq. 4 as the paper prints it, with
 * Q in R^{m x d}): chunked prefill, or verification of m speculated tokens, over a compressed cache.  For
 * every sequence b, query head hq (KV head h = hq / (Hq/Hkv)) and query i:
 *     x_t = scale * <q_i, k_hat_t> + ln(count_t),  out_i = sum_t softmax(x)_t * v_hat_t
 * over the rows t the query attends to: all t < core_len[b, h], or, with SC_FLAG_CAUSAL_TAIL, only
 * t < core_len[b, h] - (m - 1 - i) (the cache then already holds the m queries' own tokens as its last m
 * rows, stored with count 1, and each query sees itself and what precedes it).  A query that attends to
 * no row gets zeros.  With m = 1 this is sc_decode_attn.
 * The G*m query rows that share a KV head are one dense contraction against that head's cores: SC_BF16
 * with d = 128 runs on the tensor cores (scores and accumulators in tensor memory), other types and
 * head sizes on a CUDA-core kernel.  With few query rows the keys of a head are shared out among the blocks
 * of a thread-block cluster, which combine their partial results on chip.  No workspace.
 *
 *   q, out     [B, Hq, m, d] contiguous, dtype dt
 *   core_k/v, count (or NULL for all ones), cap, core_len, scale   as for sc_decode_attn
 *   flags      SC_FLAG_CAUSAL_TAIL, SC_FLAG_GENERIC (forces the CUDA-core kernel), or 0
 *   status     SC_ERR_TIMEOUT if a bounded wait inside the kernel gave up
 */
SC_API sc_status sc_prefill_attn(const void* q, sc_dtype dt, int32_t B, int32_t Hq, int32_t Hkv, int32_t m, int32_t d,
                          const void* core_k, const void* core_v, const int32_t* count, int32_t cap,
                          const int32_t* core_len, float scale, uint32_t flags, void* out,
                          int32_t* status, void* stream);

/*
 * One generated token joins a layer's compressed cache (incremental form of Sec. 2.2-2.4).
 *
 * The paper compresses the prompt's cache once and is silent about the tokens generated after
 * it.  This library's reading: the chunking rule of Eq. 1 keeps running over the generated
 * stream, starting afresh behind the prompt.  Rows [0, core_len) of a head are finished cores;
 * behind them sit tail_len tokens of the chunk that is still open, stored as they are with
 * count 1.  A call adds one token per sequence:
 *   - a token that is not a delimiter is stored behind the tail; when the tail thereby reaches
 *     max_chunk_len tokens the chunk is finished;
 *   - a delimiter finishes the open chunk (if any) and then becomes a core of its own with
 *     count 1 and its K/V bits unchanged.
 * A finished chunk is clustered (Algorithm 1 on Eq. 2) and mean-pooled (Eq. 3) where it lies,
 * its cores replacing its first rows, with the arithmetic of sc_compress's generic kernels (Sim as
 * the quotient of Eq. 2, fp32 sums in token order, one divide, one rounding; the fused bf16 path of
 * sc_compress decides G > tau*|k_i|*|k_j| and multiplies by 1/|S|, so the two can differ by one unit
 * in the last place of a core and on pairs within rounding of tau); core_len grows by the number of
 * clusters and tail_len returns to 0.  The cache therefore ends up, within the storage type's
 * tolerance, as if the generated tokens had been a second prompt.
 *
 *   k_new, v_new  [B, Hkv, d] contiguous, dtype dt: this layer's K/V of the new tokens
 *   token_ids     [B] int32 (device): the new token of each sequence
 *   delim_ids     HOST, n_delim <= SC_MAX_DELIMS ids;  max_chunk_len in [1, SC_MAX_CHUNK_LEN]
 *   tau           threshold of Algorithm 1 (Sim > tau joins)
 *   core_k/v, count, cap   the layer's cache as written by sc_compress, updated in place
 *   core_len      in/out [B, Hkv]: finished cores of each head
 *   tail_len      in/out [B, Hkv]: tokens of the open chunk (zero it once after sc_compress)
 *   attn_len      out [B, Hkv]: core_len + tail_len, the length to give sc_decode_attn
 *   status        SC_ERR_CAPACITY if a head has no free row (core_len + tail_len == cap): that
 *                 head is left as it is.  SC_ERR_INVALID_ARG for lengths that cannot be a state
 *                 of this call (negative, or tail_len >= max_chunk_len).
 * Any d > 0.  One kernel launch; no workspace.
 */
SC_API sc_status sc_append(const void* k_new, const void* v_new, sc_dtype dt, int32_t B, int32_t Hkv, int32_t d,
                    const int32_t* token_ids, const int32_t* delim_ids /*HOST*/, int32_t n_delim,
                    int32_t max_chunk_len, float tau, void* core_k, void* core_v, int32_t* count, int32_t cap,
                    int32_t* core_len, int32_t* tail_len, int32_t* attn_len, int32_t* status, void* stream);

/*
 * sc_append for every layer of a model in one launch (same reading, same arithmetic, same results).
 * For loops that have the new token's K/V of all layers at hand before the caches are updated --
 * accepting speculated tokens after verification, replaying a stored stream, a pipeline that defers
 * cache maintenance to the end of a step -- one call per generated token replaces L of them.
 *
 *   layers     DEVICE array of L rows; row l holds the pointers sc_append takes for layer l
 *              (k_new, v_new: [B, Hkv, d]; core_k, core_v, count, core_len, tail_len, attn_len as
 *              there).  The table is read by the kernel, so it may be filled once and reused as long
 *              as the buffers stay where they are.  Layers must not share any buffer.
 *   L          1..65535;  all layers share dt, B, Hkv, d, cap, token_ids, the delimiter set,
 *              max_chunk_len and tau
 *   status     as for sc_append (first error of any layer wins)
 */
typedef struct {
    const void* k_new; const void* v_new;
    void* core_k; void* core_v; int32_t* count;
    int32_t* core_len; int32_t* tail_len; int32_t* attn_len;
} sc_append_layer;

SC_API sc_status sc_append_layers(const sc_append_layer* layers /*DEVICE [L]*/, int32_t L, sc_dtype dt, int32_t B, int32_t Hkv,
                           int32_t d, const int32_t* token_ids, const int32_t* delim_ids /*HOST*/, int32_t n_delim,
                           int32_t max_chunk_len, float tau, int32_t cap, int32_t* status, void* stream);

/*
 * sc_decode_attn for callers that cannot allocate device memory.  (A convenience of this
 * library; the paper has no counterpart.)
 *
 * Who needs it: a server that handed all free HBM to its KV-cache pool at start-up, so that any
 * later cudaMalloc fails; a plug-in whose host runtime forbids allocation inside its step
 * callback; a loop that cannot tolerate the device-wide synchronisation an allocation may
 * bring.  Such callers have nowhere to get the workspace sc_decode_attn asks for.
 *
 * Same arguments, results and error codes as sc_decode_attn, minus the workspace: the split
 * partials and arrival counters live in a fixed array of SC_STATIC_SCRATCH_BYTES that is part of
 * the library image.  Every GPU on which the library is loaded holds that array until the
 * process exits, whether or not this entry point is ever called.  The call itself performs no
 * cudaMalloc / cudaFree and calls no allocating routine.
 *
 *   - Shapes whose workspace (sc_decode_workspace_bytes) exceeds SC_STATIC_SCRATCH_BYTES are
 *     rejected with SC_ERR_CAPACITY before anything is enqueued; use sc_decode_attn for those.
 *     For d = 128 the limit admits B * Hq * min(64, ceil(cap / 512)) up to about 16000, e.g.
 *     16 sequences of 32 query heads with 8K rows of capacity each.
 *   - The first call on each GPU looks up the array's device address (a short host-side set-up,
 *     done with that GPU current).  Make that first call outside any stream capture.
 *   - All calls on a GPU share the one array, which keeps the previous call's contents; each
 *     call clears the part it uses, in stream order, before its kernel runs.  Two calls that may
 *     execute concurrently on the same GPU (different streams, or SC_FLAG_OVERLAP_PREV, which is
 *     refused here with SC_ERR_INVALID_ARG) would race on it: keep them on one stream.
 */
#define SC_STATIC_SCRATCH_BYTES (8u << 20)

SC_API sc_status sc_decode_attn_static(const void* q, sc_dtype dt, int32_t B, int32_t Hq, int32_t Hkv, int32_t d,
                                const void* core_k, const void* core_v, const int32_t* count, int32_t cap,
                                const int32_t* core_len, float scale, uint32_t flags, void* out,
                                int32_t* status, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* SEMANTICACHE_H_ */
