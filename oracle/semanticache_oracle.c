/*
 * SemantiCache oracle -- TEST INFRASTRUCTURE, not the product.
 *
 * A plain, slow, obviously-correct CPU statement of what the hot path computes,
 * written from the paper's equations and Algorithm 1.  Double accumulators, no
 * blocking, no fusion, no reordering.  Nothing here is shared with the CUDA
 * path; only tests, the smoke check and the benchmark's cpu-baseline leg call it.
 *
 *   oracle_chunk   Sec. 2.2, Eq. 1     delimiter-bounded chunking
 *   oracle_gsc     Sec. 2.3, Eq. 2 + Algorithm 1   greedy seed-based clustering
 *   oracle_merge   Sec. 2.4, Eq. 3     mean-pool each cluster into a semantic core
 *   oracle_attn    Sec. 2.4, Eq. 4     proportional attention over the cores (one query per head)
 *   oracle_attn_multi  Sec. 2.4, Eq. 4 as printed (Q in R^{m x d}): a block of queries per head
 * The front end (__init__.py) adds, on top of these: the incremental path, the "no chunking" ablation
 * arm of Table 4a (oracle_gsc with one chunk per sequence) and the budget search (Table 1 budgets).
 *
 * Pins (all in tests/, none re-types these formulas): hand-worked fixtures with
 * angles whose cosines are known in closed form, the lexicographically-first
 * maximal independent set found by brute force over all subsets, partition
 * invariants, tau >= 1 reducing Eq. 4 to textbook softmax attention (numpy),
 * a cluster of identical (k, v) reproducing uncompressed attention, one query
 * of a block being the decode step, and a closed-form kept fraction on pairs at
 * known angles for the budget search.
 * The paper prints no worked numeric example, so the whole path against printed
 * values is "parity unpinned"; every function below has at least one of the pins
 * above.
 *
 * Data types: dtype 0 = bfloat16 (uint16 storage), dtype 1 = float32.
 * Tensors K, V: [B, Hkv, n, d] addressed with element strides (sb, sh, sn), the
 * last axis contiguous.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------ bf16 */

static double load_elem(const void *base, int dtype, int64_t idx) {
    if (dtype == 0) {
        uint32_t bits = ((uint32_t)((const uint16_t *)base)[idx]) << 16;
        float f;
        memcpy(&f, &bits, 4);
        return (double)f;
    }
    return (double)((const float *)base)[idx];
}

/* Round a double to the nearest bfloat16 (8 significant bits), ties to even. */
static uint16_t f64_to_bf16(double x) {
    if (isnan(x)) return 0x7fc0;
    if (x == 0.0) return signbit(x) ? 0x8000 : 0x0000;
    if (isinf(x)) return signbit(x) ? 0xff80 : 0x7f80;
    int e;
    double m = frexp(x, &e);          /* x = m * 2^e, 0.5 <= |m| < 1 */
    double r;
    if (e - 1 < -126) {               /* subnormal: fixed quantum 2^-133 */
        r = nearbyint(ldexp(x, 133)); /* default rounding mode = nearest even */
        r = ldexp(r, -133);
    } else {
        r = nearbyint(ldexp(m, 8));   /* 8 significant bits */
        r = ldexp(r, e - 8);
    }
    float f = (float)r;               /* exact: r has <= 8 significant bits */
    if (isinf(f) || fabs(r) > 3.3895313892515355e38) return signbit(x) ? 0xff80 : 0x7f80;
    uint32_t bits;
    memcpy(&bits, &f, 4);
    return (uint16_t)(bits >> 16);
}

static void store_elem(void *base, int dtype, int64_t idx, double x) {
    if (dtype == 0) ((uint16_t *)base)[idx] = f64_to_bf16(x);
    else ((float *)base)[idx] = (float)x;
}

/* exposed so a test can pin the rounding against a library conversion */
uint16_t oracle_f64_to_bf16(double x) { return f64_to_bf16(x); }

/* --------------------------------------------------------------- chunking */

static int is_delim(int32_t id, const int32_t *delim, int n_delim) {
    for (int i = 0; i < n_delim; ++i)
        if (delim[i] == id) return 1;
    return 0;
}

/*
 * Sec. 2.2, Eq. 1: split each sequence into (C_1, d_1, C_2, d_2, ..., C_M).
 * Output is an ordered list of segments over the flattened [B*n] token axis:
 * every maximal run of non-delimiter tokens is a segment (cut every
 * max_chunk_len tokens if longer), every delimiter token is a segment of length
 * one (its K/V is kept unmodified: a one-token chunk clusters to itself), empty
 * runs emit nothing, and no segment spans two sequences.
 *
 * seg_off must hold B*n+1 entries, seq_seg_off B+1.  Returns the segment count.
 */
int64_t oracle_chunk(const int32_t *token_ids, int32_t B, int32_t n,
                     const int32_t *delim, int32_t n_delim, int32_t max_chunk_len,
                     int32_t *seg_off, int32_t *seq_seg_off) {
    int64_t n_seg = 0;
    for (int32_t b = 0; b < B; ++b) {
        seq_seg_off[b] = (int32_t)n_seg;
        int32_t run = 0; /* length of the open non-delimiter run */
        for (int32_t t = 0; t < n; ++t) {
            int64_t pos = (int64_t)b * n + t;
            if (is_delim(token_ids[pos], delim, n_delim)) {
                seg_off[n_seg++] = (int32_t)pos; /* the delimiter, alone */
                run = 0;
            } else {
                if (run == 0) seg_off[n_seg++] = (int32_t)pos; /* a run opens */
                ++run;
                if (run == max_chunk_len) run = 0; /* hard cut of an over-long run */
            }
        }
    }
    seq_seg_off[B] = (int32_t)n_seg;
    seg_off[n_seg] = B * n;
    return n_seg;
}

/* -------------------------------------------------------------------- GSC */

static double dot_rows(const void *K, int dtype, int64_t a, int64_t b, int32_t d) {
    double s = 0.0;
    for (int32_t c = 0; c < d; ++c) s += load_elem(K, dtype, a + c) * load_elem(K, dtype, b + c);
    return s;
}

/* Eq. 2: cosine of two key rows; defined as 0 when either norm is 0. */
static double sim_rows(const void *K, int dtype, int64_t a, int64_t b, int32_t d) {
    double na = sqrt(dot_rows(K, dtype, a, a, d));
    double nb = sqrt(dot_rows(K, dtype, b, b, d));
    if (na == 0.0 || nb == 0.0) return 0.0;
    return dot_rows(K, dtype, a, b, d) / (na * nb);
}

/* exposed for the closed-form cosine pins */
double oracle_sim(const void *K, int32_t dtype, int64_t row_a, int64_t row_b, int32_t d) {
    return sim_rows(K, dtype, row_a * d, row_b * d, d);
}

/*
 * Algorithm 1 on every (b, head, segment) independently.
 * assign[b, h, t] = position t' (within the sequence) of the seed whose cluster
 * token t joined; a seed has assign == its own position.
 * min_margin (may be NULL) receives min |Sim - tau| over every comparison the
 * algorithm actually makes, so a test can tell that no decision was a near-tie.
 */
void oracle_gsc(const void *K, int32_t dtype, int64_t sb, int64_t sh, int64_t sn,
                int32_t B, int32_t Hkv, int32_t n, int32_t d,
                const int32_t *seg_off, const int32_t *seq_seg_off, float tau,
                int32_t *assign, double *min_margin) {
    double margin = INFINITY;
    const double thr = (double)tau;
#pragma omp parallel for collapse(2) reduction(min : margin) schedule(dynamic, 1)
    for (int32_t b = 0; b < B; ++b) {
        for (int32_t h = 0; h < Hkv; ++h) {
            unsigned char *assigned = (unsigned char *)malloc((size_t)n);
            int32_t *out = assign + ((int64_t)b * Hkv + h) * n;
            const int64_t base = b * sb + h * sh;
            for (int32_t s = seq_seg_off[b]; s < seq_seg_off[b + 1]; ++s) {
                const int32_t r = seg_off[s] - b * n;        /* first token of the chunk */
                const int32_t l = seg_off[s + 1] - seg_off[s]; /* its length */
                for (int32_t i = r; i < r + l; ++i) assigned[i] = 0;
                for (int32_t i = r; i < r + l; ++i) {
                    if (assigned[i]) continue;
                    assigned[i] = 1; /* i becomes the seed of a new cluster */
                    out[i] = i;
                    for (int32_t j = i + 1; j < r + l; ++j) {
                        if (assigned[j]) continue;
                        double sim = sim_rows(K, dtype, base + i * sn, base + j * sn, d);
                        double gap = fabs(sim - thr);
                        if (gap < margin) margin = gap;
                        if (sim > thr) { /* strict: equality does not merge */
                            assigned[j] = 1;
                            out[j] = i;
                        }
                    }
                }
            }
            free(assigned);
        }
    }
    if (min_margin) *min_margin = margin;
}

/* ------------------------------------------------------------------ merge */

/*
 * Eq. 3: each cluster becomes one core, k_hat = mean of member keys, v_hat = mean
 * of member values, rounded once to the storage dtype; count = |S_t|.  Cores are
 * laid out in position order of their seeds (a delimiter segment sits between the
 * chunks it separates).  core_k/core_v: [B, Hkv, cap, d]; count: [B, Hkv, cap];
 * core_len[b, h] = number of cores (also reported when it exceeds cap; rows
 * beyond cap are not written).
 */
void oracle_merge(const void *K, const void *V, int32_t dtype, int64_t sb, int64_t sh, int64_t sn,
                  int32_t B, int32_t Hkv, int32_t n, int32_t d,
                  const int32_t *assign, void *core_k, void *core_v, int32_t *count,
                  int32_t cap, int32_t *core_len) {
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int32_t b = 0; b < B; ++b) {
        for (int32_t h = 0; h < Hkv; ++h) {
            const int32_t *as = assign + ((int64_t)b * Hkv + h) * n;
            const int64_t base = b * sb + h * sh;
            const int64_t obase = ((int64_t)b * Hkv + h) * cap;
            double *sk = (double *)malloc(sizeof(double) * (size_t)d);
            double *sv = (double *)malloc(sizeof(double) * (size_t)d);
            int32_t row = 0;
            for (int32_t i = 0; i < n; ++i) {
                if (as[i] != i) continue; /* not a seed */
                for (int32_t c = 0; c < d; ++c) sk[c] = sv[c] = 0.0;
                int32_t cnt = 0;
                /* members carry the seed's index and lie at or after the seed */
                for (int32_t j = i; j < n; ++j) {
                    if (as[j] != i) continue;
                    for (int32_t c = 0; c < d; ++c) {
                        sk[c] += load_elem(K, dtype, base + j * sn + c);
                        sv[c] += load_elem(V, dtype, base + j * sn + c);
                    }
                    ++cnt;
                }
                if (row < cap) {
                    for (int32_t c = 0; c < d; ++c) {
                        store_elem(core_k, dtype, (obase + row) * d + c, sk[c] / cnt);
                        store_elem(core_v, dtype, (obase + row) * d + c, sv[c] / cnt);
                    }
                    count[obase + row] = cnt;
                }
                ++row;
            }
            core_len[(int64_t)b * Hkv + h] = row;
            free(sk);
            free(sv);
        }
    }
}

/*
 * Same as oracle_merge but bounded: members of a seed are searched only up to the
 * end of the seed's segment (what Algorithm 1 guarantees).  This is the routine
 * the timed cpu baseline uses; a test checks it equals oracle_merge.
 */
void oracle_merge_seg(const void *K, const void *V, int32_t dtype, int64_t sb, int64_t sh, int64_t sn,
                      int32_t B, int32_t Hkv, int32_t n, int32_t d,
                      const int32_t *seg_off, const int32_t *seq_seg_off,
                      const int32_t *assign, void *core_k, void *core_v, int32_t *count,
                      int32_t cap, int32_t *core_len) {
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int32_t b = 0; b < B; ++b) {
        for (int32_t h = 0; h < Hkv; ++h) {
            const int32_t *as = assign + ((int64_t)b * Hkv + h) * n;
            const int64_t base = b * sb + h * sh;
            const int64_t obase = ((int64_t)b * Hkv + h) * cap;
            double *sk = (double *)malloc(sizeof(double) * (size_t)d);
            double *sv = (double *)malloc(sizeof(double) * (size_t)d);
            int32_t row = 0;
            for (int32_t s = seq_seg_off[b]; s < seq_seg_off[b + 1]; ++s) {
                const int32_t r = seg_off[s] - b * n, e = seg_off[s + 1] - b * n;
                for (int32_t i = r; i < e; ++i) {
                    if (as[i] != i) continue;
                    for (int32_t c = 0; c < d; ++c) sk[c] = sv[c] = 0.0;
                    int32_t cnt = 0;
                    for (int32_t j = i; j < e; ++j) {
                        if (as[j] != i) continue;
                        for (int32_t c = 0; c < d; ++c) {
                            sk[c] += load_elem(K, dtype, base + j * sn + c);
                            sv[c] += load_elem(V, dtype, base + j * sn + c);
                        }
                        ++cnt;
                    }
                    if (row < cap) {
                        for (int32_t c = 0; c < d; ++c) {
                            store_elem(core_k, dtype, (obase + row) * d + c, sk[c] / cnt);
                            store_elem(core_v, dtype, (obase + row) * d + c, sv[c] / cnt);
                        }
                        count[obase + row] = cnt;
                    }
                    ++row;
                }
            }
            core_len[(int64_t)b * Hkv + h] = row;
            free(sk);
            free(sv);
        }
    }
}

/* -------------------------------------------------------------- attention */

/*
 * Eq. 4 for one decode step: for every query head hq (KV head = hq / (Hq/Hkv)),
 *   x_t = scale * <q, k_hat_t> + ln(count_t),   o = sum_t softmax(x)_t * v_hat_t
 * over the core_len[b, kvh] cores of that head.  count == NULL means all ones
 * (plain attention).  out is double [B, Hq, d]; a head with no cores gives zeros.
 */
void oracle_attn(const void *q, int32_t dtype, int32_t B, int32_t Hq, int32_t Hkv, int32_t d,
                 const void *core_k, const void *core_v, const int32_t *count, int32_t cap,
                 const int32_t *core_len, double scale, double *out) {
    const int32_t G = Hq / Hkv;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int32_t b = 0; b < B; ++b) {
        for (int32_t hq = 0; hq < Hq; ++hq) {
            const int32_t h = hq / G;
            const int32_t len = core_len[(int64_t)b * Hkv + h];
            const int64_t cbase = ((int64_t)b * Hkv + h) * cap;
            const int64_t qbase = ((int64_t)b * Hq + hq) * d;
            double *o = out + qbase;
            for (int32_t c = 0; c < d; ++c) o[c] = 0.0;
            if (len <= 0) continue;
            double *x = (double *)malloc(sizeof(double) * (size_t)len);
            double mx = -INFINITY;
            for (int32_t t = 0; t < len; ++t) {
                double s = 0.0;
                for (int32_t c = 0; c < d; ++c)
                    s += load_elem(q, dtype, qbase + c) * load_elem(core_k, dtype, (cbase + t) * d + c);
                x[t] = scale * s + (count ? log((double)count[cbase + t]) : 0.0);
                if (x[t] > mx) mx = x[t];
            }
            double denom = 0.0;
            for (int32_t t = 0; t < len; ++t) {
                x[t] = exp(x[t] - mx);
                denom += x[t];
            }
            for (int32_t t = 0; t < len; ++t) {
                double w = x[t] / denom;
                for (int32_t c = 0; c < d; ++c) o[c] += w * load_elem(core_v, dtype, (cbase + t) * d + c);
            }
            free(x);
        }
    }
}

/*
 * Eq. 4 with a block of queries (Q in R^{m x d}, the form the paper prints): for every
 * sequence b, query head hq (KV head = hq / (Hq/Hkv)) and query i of the m,
 *   x_t = scale * <q_i, k_hat_t> + ln(count_t),   o_i = sum_t softmax(x)_t * v_hat_t.
 * q and out are [B, Hq, m, d].  causal == 0: every query sees all core_len[b, kvh] rows.
 * causal != 0: the last m rows of the cache are the queries' own tokens (appended with count 1),
 * and query i sees rows t < core_len - (m - 1 - i): itself and everything before it.  A query
 * that sees no row gives zeros.
 */
void oracle_attn_multi(const void *q, int32_t dtype, int32_t B, int32_t Hq, int32_t Hkv, int32_t m, int32_t d,
                       const void *core_k, const void *core_v, const int32_t *count, int32_t cap,
                       const int32_t *core_len, double scale, int32_t causal, double *out) {
    const int32_t G = Hq / Hkv;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int32_t b = 0; b < B; ++b) {
        for (int32_t hq = 0; hq < Hq; ++hq) {
            const int32_t h = hq / G;
            const int32_t len = core_len[(int64_t)b * Hkv + h];
            const int64_t cbase = ((int64_t)b * Hkv + h) * cap;
            double *x = (double *)malloc(sizeof(double) * (size_t)(len > 0 ? len : 1));
            for (int32_t i = 0; i < m; ++i) {
                const int64_t qbase = (((int64_t)b * Hq + hq) * m + i) * d;
                double *o = out + qbase;
                for (int32_t c = 0; c < d; ++c) o[c] = 0.0;
                const int32_t vis = causal ? len - (m - 1 - i) : len; /* rows this query sees */
                if (vis <= 0) continue;
                double mx = -INFINITY;
                for (int32_t t = 0; t < vis; ++t) {
                    double s = 0.0;
                    for (int32_t c = 0; c < d; ++c)
                        s += load_elem(q, dtype, qbase + c) * load_elem(core_k, dtype, (cbase + t) * d + c);
                    x[t] = scale * s + (count ? log((double)count[cbase + t]) : 0.0);
                    if (x[t] > mx) mx = x[t];
                }
                double denom = 0.0;
                for (int32_t t = 0; t < vis; ++t) {
                    x[t] = exp(x[t] - mx);
                    denom += x[t];
                }
                for (int32_t t = 0; t < vis; ++t) {
                    double w = x[t] / denom;
                    for (int32_t c = 0; c < d; ++c) o[c] += w * load_elem(core_v, dtype, (cbase + t) * d + c);
                }
            }
            free(x);
        }
    }
}
