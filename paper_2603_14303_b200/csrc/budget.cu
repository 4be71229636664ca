// sc_compress_budget: compress a layer to a KV budget (the kept fractions of the paper's Table 1;
// Table 4b: a lower threshold keeps fewer entries).  The paper does not say how a budget becomes a
// threshold; here the threshold is searched on a grid, on the device, without a host round trip:
// a fixed sequence of counting passes (Algorithm 1 without Eq. 3, keys only) alternates with a
// one-block step kernel that adds up the cluster counts, narrows the interval and writes the next
// threshold to device memory; once the choice is made the remaining counting passes find a flag set
// and return at once, and a final ordinary compress pass runs at the chosen threshold.
#include "common.cuh"

namespace sc {

bool compress_fused_supported(const CompressArgs& a);
cudaError_t launch_compress_fused(const CompressArgs& a, cudaStream_t st);

namespace bg {

// Search state in device memory (one per workspace).
struct State {
    long long k_lo, k_hi;   // cluster counts at the interval's ends
    int lo, hi;             // grid indices: count(lo) < target <= count(hi) once both are known
    int phase;              // 0: lowest index is being counted, 1: highest, 2: a middle one
    int done;               // nonzero: `pick` is final, further counting passes do nothing
    int pick;
    int passes;             // counting passes that did work
    float tau;              // threshold of the pass in flight, then the chosen one
};

struct Grid { float tau[SC_BUDGET_MAX_GRID]; };

__global__ void budget_init(State* s, int32_t* core_len, int heads, int n_grid, Grid g) {
    for (int i = threadIdx.x; i < heads; i += blockDim.x) core_len[i] = 0;
    if (threadIdx.x == 0) {
        s->k_lo = s->k_hi = 0;
        s->lo = 0; s->hi = n_grid - 1;
        s->phase = 0; s->done = 0; s->pick = 0; s->passes = 0;
        s->tau = g.tau[0];
    }
}

// After a counting pass: total the per-head counts (and clear them for the next pass), move the search on.
__global__ void __launch_bounds__(256)
budget_step(State* s, int32_t* core_len, int heads, long long target, Grid g, float* tau_out, int32_t* search_out) {
    __shared__ long long part[8];
    if (s->done) return;   // the choice was made earlier: the pass before this step did nothing
    long long sum = 0;
    for (int i = threadIdx.x; i < heads; i += blockDim.x) {
        sum += core_len[i];
        core_len[i] = 0;
    }
    for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(kFull, sum, o);
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = sum;
    __syncthreads();
    if (threadIdx.x != 0) return;
    long long k = 0;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) k += part[w];
    int lo = s->lo, hi = s->hi, pick = -1;
    s->passes += 1;
    if (s->phase == 0) {
        s->k_lo = k;
        if (k >= target || hi == lo) pick = lo;   // even the lowest threshold keeps at least the target
        else { s->phase = 1; s->tau = g.tau[hi]; }
    } else {
        if (s->phase == 1) {
            s->k_hi = k;
            if (k < target) pick = hi;            // even the highest threshold keeps less than the target
            s->phase = 2;
        } else {
            const int mid = (lo + hi) / 2;
            if (k >= target) { hi = mid; s->k_hi = k; } else { lo = mid; s->k_lo = k; }
            s->lo = lo; s->hi = hi;
        }
        if (pick < 0) {
            if (hi - lo > 1) s->tau = g.tau[(lo + hi) / 2];
            else pick = (s->k_hi - target) < (target - s->k_lo) ? hi : lo;   // the nearer end, the lower on a tie
        }
    }
    if (pick >= 0) {
        s->pick = pick; s->done = 1; s->tau = g.tau[pick];
        if (tau_out) *tau_out = g.tau[pick];
        if (search_out) { search_out[0] = pick; search_out[1] = s->passes; }
    }
}

}  // namespace bg

size_t budget_state_bytes() { return (sizeof(bg::State) + 255) / 256 * 256; }

// `a` is a complete sc_compress argument set whose workspace starts with budget_state_bytes() for the
// search state; `ws_compress` / `ws_generic` are the fused kernel's and the generic kernels' regions behind it.
cudaError_t launch_compress_budget(CompressArgs a, void* ws_compress, void* ws_generic, const float* grid, int n_grid,
                                   long long target, float* tau_out, int32_t* search_out, cudaStream_t st) {
    bg::State* state = (bg::State*)a.ws;
    bg::Grid g;
    for (int i = 0; i < SC_BUDGET_MAX_GRID; ++i) g.tau[i] = grid[i < n_grid ? i : n_grid - 1];
    const int heads = a.B * a.Hkv;
    int passes = 2;
    for (int span = n_grid - 1; span > 1; span = (span + 1) / 2) ++passes;   // 2 + ceil(log2(n_grid - 1))
    if (n_grid <= 2) passes = n_grid;
    bg::budget_init<<<1, 256, 0, st>>>(state, a.core_len, heads, n_grid, g);
    note_launches(1);
    bool fused = !(a.flags & SC_FLAG_GENERIC) && compress_fused_supported(a);
    CompressArgs c = a;
    c.tau_dev = &state->tau; c.skip = &state->done; c.count_only = 1; c.assign = nullptr;
    for (int p = 0; p < passes; ++p) {
        cudaError_t e = cudaErrorNotSupported;
        if (fused) { c.ws = ws_compress; e = launch_compress_fused(c, st); }
        if (e == cudaErrorNotSupported) { fused = false; c.ws = ws_generic; e = launch_compress_generic(c, st); }
        if (e != cudaSuccess) return e;
        bg::budget_step<<<1, 256, 0, st>>>(state, a.core_len, heads, target, g, tau_out, search_out);
        note_launches(1);
    }
    // the pass that writes the cores, at the chosen threshold
    CompressArgs f = a;
    f.tau_dev = &state->tau; f.skip = nullptr; f.count_only = 0;
    cudaError_t e = cudaErrorNotSupported;
    if (fused) { f.ws = ws_compress; e = launch_compress_fused(f, st); }
    if (e == cudaErrorNotSupported) { f.ws = ws_generic; e = launch_compress_generic(f, st); }
    return e;
}

}  // namespace sc
