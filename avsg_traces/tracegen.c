/*
 * Seeded synthetic inputs for the AVSG per-decode-step operator: DSA-style
 * top-K selection traces and host KV bytes.
 *
 * This file only DRAWS inputs.  It contains none of the operator's arithmetic
 * (no matching, no lifetimes, no slot allocation, no gather); both the CPU
 * oracle's tests and the CUDA path's tests feed on what it produces.
 *
 * Randomness: splitmix64.  A trace uses one sequential stream per
 * (seed, table); host KV bytes are a stateless hash of (seed, table, word
 * index), so any row can be recomputed without storing a second copy.
 *
 * Trace recipe for one table (T iterations of N_q query tokens, K ids each):
 *   query tokens are numbered q = t*N_q + g;
 *   q == 0 : K distinct ids uniform over [0, lim(q));
 *   q  > 0 : keep = floor(rho*K) ids drawn without replacement from the
 *            selection of token q-1, the remaining K-keep ids drawn by
 *            rejection (distinct from everything already chosen) from a
 *            mixture of {recent window, fixed hot set, history of earlier
 *            selections, uniform};
 *   every selection is emitted sorted ascending, padded with -1 when the
 *   drawable range holds fewer than K ids.
 *   lim(q) = verified_len(t) + g, with verified_len(t) = context -
 *   N_q*(T - t) when the context grows (all speculative tokens accepted), or
 *   lim(q) = verified_len(t) = context when it does not.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef struct {
    uint64_t seed;
    uint32_t table;         /* stream id: one independent stream per table   */
    uint32_t topk;          /* K                                             */
    uint32_t n_q;           /* query tokens per iteration                    */
    uint32_t n_iters;       /* T                                             */
    int64_t  context;       /* context length at the END of the trace        */
    int32_t  ctx_growth;    /* 1: verified length grows by n_q per iteration */
    int32_t  rho_kind;      /* 0: fixed rho, 1: Beta(beta_a, beta_b)         */
    double   rho_fixed;
    int32_t  beta_a, beta_b;
    double   p_recent;      /* share of new ids drawn from the recent window */
    uint32_t recent_window;
    double   p_hot;         /* share of new ids drawn from the hot set       */
    uint32_t hot_size;      /* ids in the per-table hot set                  */
    uint32_t hot_range;     /* hot ids are distinct draws from [0,hot_range) */
    double   p_hist;        /* share of new ids drawn from ids selected at any
                               earlier step ("historical recall")            */
    double   hist_sigma;    /* p_hist is redrawn per token as N(p_hist, sigma^2)
                               clipped to [0,1] when sigma > 0               */
} tg_config;

static inline uint64_t sm64_next(uint64_t *s)
{
    uint64_t z = (*s += 0x9E3779B97F4A7C15ull);
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

static inline uint64_t sm64_hash(uint64_t key)
{
    uint64_t s = key;
    return sm64_next(&s);
}

static inline double u01(uint64_t *s)
{
    return (double)(sm64_next(s) >> 11) * (1.0 / 9007199254740992.0);
}

static inline uint64_t below(uint64_t *s, uint64_t n)
{
    return sm64_next(s) % n;
}

static int cmp_i32(const void *a, const void *b)
{
    int32_t x = *(const int32_t *)a, y = *(const int32_t *)b;
    return (x > y) - (x < y);
}

static int cmp_f64(const void *a, const void *b)
{
    double x = *(const double *)a, y = *(const double *)b;
    return (x > y) - (x < y);
}

/* Beta(a,b) for integer a,b >= 1: the a-th smallest of a+b-1 uniforms. */
static double beta_int(uint64_t *s, int a, int b)
{
    double u[64];
    int n = a + b - 1;
    if (n > 64) n = 64;
    for (int i = 0; i < n; ++i) u[i] = u01(s);
    qsort(u, (size_t)n, sizeof(double), cmp_f64);
    return u[a - 1];
}

uint64_t tg_stream_seed(uint64_t seed, uint32_t table)
{
    return sm64_hash(seed ^ ((uint64_t)table << 40) ^ 0x7472616365ull);
}

/* Verified context length of iteration t (what the operator is told). */
int32_t tg_verified_len(const tg_config *c, uint32_t t)
{
    if (!c->ctx_growth) return (int32_t)c->context;
    return (int32_t)(c->context - (int64_t)c->n_q * (int64_t)(c->n_iters - t));
}

/*
 * Writes X[T][N_q][K] (int32, ascending, -1 padded) and verified_len[T].
 * Returns 0, or -1 on a bad configuration / allocation failure.
 */
int tg_generate(const tg_config *c, int32_t *X, int32_t *verified_len)
{
    const uint32_t K = c->topk;
    if (K == 0 || c->n_q == 0 || c->n_iters == 0 || c->context <= 0) return -1;
    if (c->ctx_growth && c->context - (int64_t)c->n_q * c->n_iters <= 0) return -1;
    if (c->context > 0x7fffffff) return -1;

    uint64_t s = tg_stream_seed(c->seed, c->table);
    uint8_t *mark = (uint8_t *)calloc((size_t)c->context + c->n_q + 1, 1);
    int32_t *prev = (int32_t *)malloc(sizeof(int32_t) * K);
    int32_t *cur = (int32_t *)malloc(sizeof(int32_t) * K);
    int32_t *hot = c->hot_size ? (int32_t *)malloc(sizeof(int32_t) * c->hot_size) : NULL;
    /* history: every id selected so far, each once (seen[] marks membership) */
    const int use_hist = c->p_hist > 0.0;
    int32_t *hist = use_hist ? (int32_t *)malloc(sizeof(int32_t) * ((size_t)c->context + c->n_q + 1)) : NULL;
    uint8_t *seen = use_hist ? (uint8_t *)calloc((size_t)c->context + c->n_q + 1, 1) : NULL;
    size_t n_hist = 0;
    if (!mark || !prev || !cur || (c->hot_size && !hot) || (use_hist && (!hist || !seen))) {
        free(mark); free(prev); free(cur); free(hot); free(hist); free(seen);
        return -1;
    }

    /* fixed per-table hot set: hot_size distinct ids from [0, hot_range) */
    uint32_t n_hot = 0;
    if (c->hot_size) {
        uint32_t range = c->hot_range;
        if (range < c->hot_size) range = c->hot_size;
        while (n_hot < c->hot_size) {
            int32_t id = (int32_t)below(&s, range);
            if (!mark[id]) { mark[id] = 1; hot[n_hot++] = id; }
        }
        for (uint32_t i = 0; i < n_hot; ++i) mark[hot[i]] = 0;
    }

    uint32_t n_prev = 0;
    for (uint32_t t = 0; t < c->n_iters; ++t) {
        const int64_t N = tg_verified_len(c, t);
        verified_len[t] = (int32_t)N;
        for (uint32_t g = 0; g < c->n_q; ++g) {
            const int64_t lim = c->ctx_growth ? N + g : N;
            const uint32_t want = (lim < (int64_t)K) ? (uint32_t)lim : K;
            uint32_t n_cur = 0;

            if (t > 0 || g > 0) {
                double rho = c->rho_kind ? beta_int(&s, c->beta_a, c->beta_b) : c->rho_fixed;
                uint32_t keep = (uint32_t)floor(rho * (double)K);
                if (keep > n_prev) keep = n_prev;
                if (keep > want) keep = want;
                /* partial Fisher-Yates over the previous selection */
                for (uint32_t i = 0; i < keep; ++i) {
                    uint32_t j = i + (uint32_t)below(&s, n_prev - i);
                    int32_t tmp = prev[i]; prev[i] = prev[j]; prev[j] = tmp;
                    cur[n_cur++] = prev[i];
                    mark[prev[i]] = 1;
                }
            }
            double p_hist = c->p_hist;
            if (use_hist && c->hist_sigma > 0.0) {      /* Box-Muller normal, clipped to [0,1] */
                double u1 = u01(&s), u2 = u01(&s);
                if (u1 < 1e-300) u1 = 1e-300;
                p_hist += c->hist_sigma * sqrt(-2.0 * log(u1)) * cos(6.283185307179586 * u2);
                if (p_hist < 0.0) p_hist = 0.0;
                if (p_hist > 1.0) p_hist = 1.0;
            }
            while (n_cur < want) {
                int32_t id = -1;
                double comp = u01(&s);
                if (use_hist && comp < p_hist && n_hist) {
                    for (int tries = 0; tries < 64; ++tries) {
                        int32_t cand = hist[below(&s, n_hist)];
                        if (cand < lim && !mark[cand]) { id = cand; break; }
                    }
                    comp = 2.0;                          /* the other restricted components are skipped */
                }
                if (id >= 0) {
                    /* drawn from history */
                } else if (comp < c->p_recent && c->recent_window) {
                    int64_t w = c->recent_window < lim ? c->recent_window : lim;
                    for (int tries = 0; tries < 64; ++tries) {
                        int32_t cand = (int32_t)(lim - 1 - (int64_t)below(&s, (uint64_t)w));
                        if (!mark[cand]) { id = cand; break; }
                    }
                } else if (comp < c->p_recent + c->p_hot && n_hot) {
                    for (int tries = 0; tries < 64; ++tries) {
                        int32_t cand = hot[below(&s, n_hot)];
                        if (cand < lim && !mark[cand]) { id = cand; break; }
                    }
                }
                while (id < 0) {   /* uniform component and fall-back */
                    int32_t cand = (int32_t)below(&s, (uint64_t)lim);
                    if (!mark[cand]) id = cand;
                }
                mark[id] = 1;
                cur[n_cur++] = id;
            }
            for (uint32_t i = 0; i < n_cur; ++i) mark[cur[i]] = 0;
            if (use_hist)
                for (uint32_t i = 0; i < n_cur; ++i)
                    if (!seen[cur[i]]) { seen[cur[i]] = 1; hist[n_hist++] = cur[i]; }
            qsort(cur, n_cur, sizeof(int32_t), cmp_i32);

            int32_t *out = X + ((size_t)t * c->n_q + g) * K;
            memcpy(out, cur, sizeof(int32_t) * n_cur);
            for (uint32_t i = n_cur; i < K; ++i) out[i] = -1;
            memcpy(prev, cur, sizeof(int32_t) * n_cur);
            n_prev = n_cur;
        }
    }
    free(mark); free(prev); free(cur); free(hot); free(hist); free(seen);
    return 0;
}

/* Host KV: 8-byte word w of a table is a hash of (seed, table, w). */
static inline uint64_t kv_word(uint64_t key, uint64_t w)
{
    return sm64_hash(key + w * 0xD1342543DE82EF95ull);
}

static inline uint64_t kv_key(uint64_t seed, uint32_t table)
{
    return sm64_hash(seed ^ ((uint64_t)table << 40) ^ 0x6b76ull);
}

/*
 * Fills rows [first_row, first_row + n_rows) of one table's host KV.
 * dst points at the first of those rows; rows are row_stride bytes apart and
 * carry row_bytes (multiple of 8) payload bytes; bytes between payload and
 * stride are left untouched.  Row content depends on (seed, table, row,
 * version) only; version lets a test "regenerate" a row with other bytes.
 */
void tg_fill_kv(uint8_t *dst, uint64_t seed, uint32_t table, uint64_t first_row,
                uint64_t n_rows, uint32_t row_bytes, uint64_t row_stride, uint32_t version)
{
    const uint64_t key = kv_key(seed, table) ^ ((uint64_t)version * 0xA24BAED4963EE407ull);
    const uint64_t wpr = row_bytes / 8;
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < (int64_t)n_rows; ++r) {
        uint64_t *row = (uint64_t *)(dst + (uint64_t)r * row_stride);
        const uint64_t w0 = (first_row + (uint64_t)r) * wpr;
        for (uint64_t w = 0; w < wpr; ++w) row[w] = kv_word(key, w0 + w);
    }
}

/* log-uniform integer in [lo, hi] and uniform double in [a, b): per-table
 * parameters of the load-imbalance configuration. */
int64_t tg_log_uniform(uint64_t seed, uint32_t table, int64_t lo, int64_t hi)
{
    uint64_t s = sm64_hash(seed ^ ((uint64_t)table << 40) ^ 0x63747874ull);
    double u = u01(&s);
    double v = exp(log((double)lo) + u * (log((double)hi) - log((double)lo)));
    int64_t r = (int64_t)floor(v);
    if (r < lo) r = lo;
    if (r > hi) r = hi;
    return r;
}

double tg_uniform(uint64_t seed, uint32_t table, double a, double b)
{
    uint64_t s = sm64_hash(seed ^ ((uint64_t)table << 40) ^ 0x72686f6full);
    return a + (b - a) * u01(&s);
}

/* Recomputes an arbitrary list of rows (packed, row_bytes apart) of one table. */
void tg_kv_rows(uint8_t *dst, uint64_t seed, uint32_t table, const int64_t *rows,
                uint64_t n, uint32_t row_bytes, uint32_t version)
{
    const uint64_t key = kv_key(seed, table) ^ ((uint64_t)version * 0xA24BAED4963EE407ull);
    const uint64_t wpr = row_bytes / 8;
    for (uint64_t r = 0; r < n; ++r) {
        uint64_t *row = (uint64_t *)(dst + r * (uint64_t)row_bytes);
        const uint64_t w0 = (uint64_t)rows[r] * wpr;
        for (uint64_t w = 0; w < wpr; ++w) row[w] = kv_word(key, w0 + w);
    }
}
