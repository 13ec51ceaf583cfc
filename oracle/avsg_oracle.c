/*
 * CPU oracle of the AVSG per-decode-step operator.
 *
 * TEST INFRASTRUCTURE ONLY.  Plain, slow, single-threaded C that restates the
 * paper's algorithms step by step so that a reader can check it against the
 * paper by eye.  It shares no code with the CUDA path and the product never
 * calls it; tests, the smoke check and the benchmark's CPU-baseline leg do.
 *
 * What is restated, and from where:
 *   - hit / miss definition ............ Eq. 1 (residency), Sec. 3.2
 *   - Stage One, three passes per token  Algorithm 1
 *   - CollectDead ...................... Eq. 12
 *   - life-cycle update ................ Algorithm 3
 *   - MTP sequencing + invalidation .... Algorithm 4
 *   - balanced miss partition .......... Eq. 6, Sec. 3.4
 *   - request-level assignment ......... Eq. 13 (comparator S1)
 *   - equal top-K position partition ... Eq. 14 (comparator S2)
 *   - paper-literal Hash-State mode .... Eq. 2-4, Eq. 8-11, Algorithm 2 (second half of this file)
 *
 * Readings taken where the paper is silent or ambiguous (all listed in the
 * design notes of the repository):
 *   - matching is EXACT residency (Eq. 1): an id hits iff some slot holds it
 *     at the moment its token is processed.  The bounded-retry hash probe of
 *     the paper's NPU kernel is an implementation of this test that may lose
 *     mappings; it is not modelled.  Matching here is a linear scan.
 *   - a lifetime is a signed counter that saturates at -1 ("dead"); dead
 *     slots stay dead however long they idle.
 *   - the table starts with every slot empty (id -1) and dead (-1).
 *   - a dead slot that still holds an id can be hit and is revived to L
 *     (Probe compares ids only).
 *   - invalidation clears the id only; the slot's lifetime is left as is.
 *   - negative ids are padding: slot -1, neither hit nor miss.
 *   - ids are unique within one token's list (precondition).
 *
 * Parity pins (tests/, marker "not gpu"): brute-force set membership, the
 * S = K special case (hits = |sel_t ∩ sel_{t-1}|), the no-pressure special
 * case (hit iff selected at any earlier step), cold start, unchanged
 * selection, MTP sharing, a hand-worked allocation example, and the
 * invariants of Sec. 3.4/3.5.  The paper prints no worked example with
 * concrete ids, so beyond those pins per-step values are "parity unpinned".
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORC_OK         0
#define ORC_EINVAL    -1
#define ORC_ECAPACITY -2   /* Eq. 7 violated: S < N_q * K */
#define ORC_ENOMEM    -3

typedef struct orc_table {
    uint32_t S;          /* slots                                            */
    uint32_t row_bytes;
    int32_t  L;          /* maximum lifetime                                 */
    int32_t *c;          /* c[j]: id cached in slot j, -1 = empty (Sec. 3.2) */
    int32_t *life;       /* lifetime of slot j; < 0 = dead (Eq. 12)          */
    uint8_t *rows;       /* S rows of row_bytes: the HBM buffer              */
    /* running counters */
    uint64_t steps, tokens, hits, misses, rows_copied, extra_decays;
} orc_table;

/* One entry of the transfer list: host position x -> device slot o. */
typedef struct { int32_t x; int32_t o; } orc_xfer;

orc_table *orc_create(uint32_t S, uint32_t row_bytes, int32_t L)
{
    if (S == 0 || L < 1 || L > 126) return NULL;
    orc_table *t = (orc_table *)calloc(1, sizeof(*t));
    if (!t) return NULL;
    t->S = S; t->row_bytes = row_bytes; t->L = L;
    t->c = (int32_t *)malloc(sizeof(int32_t) * S);
    t->life = (int32_t *)malloc(sizeof(int32_t) * S);
    t->rows = (uint8_t *)calloc((size_t)S, row_bytes ? row_bytes : 1);
    if (!t->c || !t->life || !t->rows) { free(t->c); free(t->life); free(t->rows); free(t); return NULL; }
    for (uint32_t j = 0; j < S; ++j) { t->c[j] = -1; t->life[j] = -1; }
    return t;
}

void orc_destroy(orc_table *t)
{
    if (!t) return;
    free(t->c); free(t->life); free(t->rows); free(t);
}

/* A new request finds nothing cached (App. E): every slot empty and dead, rows and counters zero. */
void orc_reset(orc_table *t)
{
    for (uint32_t j = 0; j < t->S; ++j) { t->c[j] = -1; t->life[j] = -1; }
    memset(t->rows, 0, (size_t)t->S * t->row_bytes);
    t->steps = t->tokens = t->hits = t->misses = t->rows_copied = t->extra_decays = 0;
}

/* Eq. 1: is x resident, and in which slot?  Lifetime is not consulted. */
int32_t orc_find(const orc_table *t, int32_t x)
{
    if (x < 0) return -1;
    for (uint32_t j = 0; j < t->S; ++j)
        if (t->c[j] == x) return (int32_t)j;
    return -1;
}

/* One unit decay of every lifetime (Alg. 1 line "s.lifetime <- s.lifetime - 1"),
 * saturating at -1. */
static void decay_all(orc_table *t)
{
    for (uint32_t j = 0; j < t->S; ++j)
        if (t->life[j] > -1) t->life[j] -= 1;
}

/* Eq. 12: slots with lifetime < 0, increasing order, each once. */
uint32_t orc_collect_dead(const orc_table *t, int32_t *e)
{
    uint32_t n = 0;
    for (uint32_t j = 0; j < t->S; ++j)
        if (t->life[j] < 0) e[n++] = (int32_t)j;
    return n;
}

/*
 * Algorithm 1 for token g of a request (with the lifetime operations of
 * Algorithm 3).  x[K] in; o[K], m[K] out; misses appended to list (capacity
 * >= *n_list + K).  Returns n_g, or a negative error.
 */
int32_t orc_stage_one_token(orc_table *t, uint32_t g, const int32_t *x, uint32_t K,
                            int32_t *o, uint8_t *m, orc_xfer *list, uint32_t *n_list)
{
    int32_t *e = (int32_t *)malloc(sizeof(int32_t) * t->S);
    if (!e) return ORC_ENOMEM;

    /* Pass 1 - Refresh: global pre-decay for the first token only */
    if (g == 0) decay_all(t);
    /* Probe: hit mask and hit slots (read-only) */
    for (uint32_t i = 0; i < K; ++i) {
        int32_t j = orc_find(t, x[i]);
        m[i] = (uint8_t)(j >= 0);
        o[i] = j;                       /* -1 for misses (placeholder) and padding */
    }
    /* restore the lifetime of matched entries to L, before any allocation */
    for (uint32_t i = 0; i < K; ++i)
        if (m[i]) t->life[o[i]] = t->L;

    /* Pass 2 - Classify: miss count over the valid (non-padding) ids */
    int32_t n_g = 0;
    uint32_t valid = 0;
    for (uint32_t i = 0; i < K; ++i)
        if (x[i] >= 0) { valid++; n_g += 1 - (int32_t)m[i]; }

    /* Pass 3 - Allocate */
    uint32_t n_dead = orc_collect_dead(t, e);
    while (n_dead < (uint32_t)n_g) {
        int any_alive = 0;
        for (uint32_t j = 0; j < t->S; ++j) any_alive |= (t->life[j] >= 0);
        if (!any_alive) { free(e); return ORC_ECAPACITY; }   /* cannot happen when S >= K */
        decay_all(t);
        t->extra_decays++;
        n_dead = orc_collect_dead(t, e);
    }
    /* t = x[not m] keeps order; o_miss = e[:n_g]; UpdateState writes id and lifetime */
    uint32_t k = 0;
    for (uint32_t i = 0; i < K; ++i) {
        if (x[i] < 0 || m[i]) continue;
        int32_t j = e[k++];
        t->c[j] = x[i];
        t->life[j] = t->L;
        o[i] = j;
        list[*n_list].x = x[i];
        list[*n_list].o = j;
        (*n_list)++;
    }
    t->tokens++;
    t->hits += valid - (uint32_t)n_g;
    t->misses += (uint32_t)n_g;
    free(e);
    return n_g;
}

/* Stage Two: every listed miss is copied exactly once, host row x -> slot o. */
void orc_stage_two(orc_table *t, const orc_xfer *list, uint32_t n_list,
                   const uint8_t *host_kv, uint64_t row_stride)
{
    for (uint32_t k = 0; k < n_list; ++k)
        memcpy(t->rows + (size_t)list[k].o * t->row_bytes,
               host_kv + (uint64_t)list[k].x * row_stride, t->row_bytes);
    t->rows_copied += n_list;
}

/* Algorithm 4, end of step: entries with c_j >= N become empty. */
void orc_invalidate(orc_table *t, int32_t N)
{
    for (uint32_t j = 0; j < t->S; ++j)
        if (t->c[j] >= N) t->c[j] = -1;
}

/*
 * Algorithm 4: one decode step of one request table.
 *   X[N_q][K] in; O[N_q][K], M[N_q][K], n[N_q] out;
 *   list (capacity N_q*K) receives the step's transfer list, *n_list its length.
 * host_kv may be NULL (no bytes are moved then).
 */
int orc_step(orc_table *t, const int32_t *X, uint32_t N_q, uint32_t K, int32_t N,
             const uint8_t *host_kv, uint64_t row_stride,
             int32_t *O, uint8_t *M, int32_t *n, orc_xfer *list, uint32_t *n_list)
{
    if ((uint64_t)N_q * K > t->S) return ORC_ECAPACITY;     /* Eq. 7 */
    *n_list = 0;
    for (uint32_t g = 0; g < N_q; ++g) {
        int32_t r = orc_stage_one_token(t, g, X + (size_t)g * K, K, O + (size_t)g * K,
                                        M + (size_t)g * K, list, n_list);
        if (r < 0) return r;
        n[g] = r;
    }
    if (host_kv) orc_stage_two(t, list, *n_list, host_kv, row_stride);
    orc_invalidate(t, N);
    t->steps++;
    return ORC_OK;
}

/*
 * "KV Offload" comparator (Sec. 4.1): no reuse, all N_q*K selected rows are
 * transferred every step; position (g, i) lands in slot g*K + i.
 */
int orc_step_all_k(orc_table *t, const int32_t *X, uint32_t N_q, uint32_t K,
                   const uint8_t *host_kv, uint64_t row_stride, int32_t *O)
{
    if ((uint64_t)N_q * K > t->S) return ORC_ECAPACITY;
    for (uint32_t p = 0; p < N_q * K; ++p) {
        if (X[p] < 0) { O[p] = -1; continue; }
        O[p] = (int32_t)p;
        if (host_kv)
            memcpy(t->rows + (size_t)p * t->row_bytes, host_kv + (uint64_t)X[p] * row_stride, t->row_bytes);
        t->rows_copied++;
    }
    t->steps++;
    return ORC_OK;
}

/*
 * Eq. 6: the miss list, ordered by token, is cut into C consecutive pieces of
 * floor(N/C) or ceil(N/C) entries; the first N mod C cores take the larger
 * share.  Returns core c's range [begin, end).
 */
void orc_partition(uint64_t n_miss, uint32_t C, uint32_t c, uint64_t *begin, uint64_t *end)
{
    uint64_t q = n_miss / C, r = n_miss % C;
    *begin = (uint64_t)c * q + (c < r ? c : r);
    *end = *begin + q + (c < r ? 1 : 0);
}

/* Eq. 13: request-level assignment; core c serves requests c, c + C, ...
 * (first B mod C cores take one extra request).  Returns how many. */
uint32_t orc_requests_of_core(uint32_t B, uint32_t C, uint32_t c)
{
    return B / C + (c < B % C ? 1u : 0u);
}

/* Eq. 14: equal top-K position partitioning; core c takes the flattened
 * positions floor(c*NgK/C) <= gK+i < floor((c+1)*NgK/C), hits included. */
void orc_position_range(uint64_t n_positions, uint32_t C, uint32_t c, uint64_t *begin, uint64_t *end)
{
    *begin = (uint64_t)c * n_positions / C;
    *end = (uint64_t)(c + 1) * n_positions / C;
}

/* Eq. 5: transfer workload of a set of positions = the misses among them.
 * m[] is the hit mask over the flattened positions; padding counts as no work. */
uint64_t orc_workload(const uint8_t *m, const int32_t *x, uint64_t begin, uint64_t end)
{
    uint64_t w = 0;
    for (uint64_t p = begin; p < end; ++p)
        if (x[p] >= 0) w += 1u - m[p];
    return w;
}

/* accessors for the Python test harness */
uint32_t orc_slots(const orc_table *t) { return t->S; }
void orc_export(const orc_table *t, int32_t *c, int8_t *life)
{
    for (uint32_t j = 0; j < t->S; ++j) { c[j] = t->c[j]; life[j] = (int8_t)t->life[j]; }
}
void orc_import(orc_table *t, const int32_t *c, const int8_t *life)
{
    for (uint32_t j = 0; j < t->S; ++j) { t->c[j] = c[j]; t->life[j] = life[j]; }
}
const uint8_t *orc_rows(const orc_table *t) { return t->rows; }
void orc_counters(const orc_table *t, uint64_t out[6])
{
    out[0] = t->steps; out[1] = t->tokens; out[2] = t->hits;
    out[3] = t->misses; out[4] = t->rows_copied; out[5] = t->extra_decays;
}

/* ==========================================================================
 * Paper-literal Hash-State mode (Sec. 3.2-3.3, App. B).
 *
 * The table is S 64-bit entries E_j = (c_j, q_j); q_j packs, from the most
 * significant bit: lifetime (8, signed) | invalid (1) | fingerprint (23-m) |
 * slot (m), S = 2^m (Eq. 2).  The lifetime belongs to SLOT j, the low 24 bits
 * are BUCKET j's mapping.  Probing is bounded (R + 1 buckets, Eq. 8-11) and a
 * bucket's mapping can be overwritten by another id (Alg. 2), so a resident id
 * can be missed and fetched again: this mode is lossy by design and does not
 * compute Eq. 1 exactly.
 *
 * Readings needed to make it deterministic (the paper leaves them open):
 *   - a1, a2 are parameters (two distinct odd primes);
 *   - when several misses of one token write the same bucket word, the paper
 *     lets an unspecified one of them win (Alg. 2): here the miss with the
 *     HIGHEST position wins;
 *   - Alg. 2 evaluates all probes on the table as it is when UpdateState is
 *     entered, then writes ids and lifetimes, then writes the bucket words,
 *     reading the preserved lifetime at that moment (statement order);
 *   - lifetime saturates at -1; initial word: lifetime -1, invalid 1;
 *   - phi(c) of an empty slot (c = -1) is taken on the unsigned value.
 * Beyond its own invariants (tests) this mode is "parity unpinned".
 * ========================================================================== */
typedef struct orc_lit_table {
    uint32_t S, m, row_bytes, R;
    int32_t  L;
    uint32_t a1, a2;
    int32_t  *c;
    uint32_t *q;
    uint8_t  *rows;
    uint64_t steps, tokens, hits, misses, rows_copied, extra_decays, lost_mappings;
} orc_lit_table;

static int32_t lit_life(uint32_t q) { return (int32_t)(int8_t)(q >> 24); }
static uint32_t lit_set_life(uint32_t q, int32_t l) { return (q & 0x00FFFFFFu) | ((uint32_t)(uint8_t)(int8_t)l << 24); }

orc_lit_table *orc_lit_create(uint32_t S, uint32_t row_bytes, int32_t L, uint32_t R, uint32_t a1, uint32_t a2)
{
    uint32_t m = 0;
    while ((1u << m) < S) ++m;
    if (S < 2 || (1u << m) != S || m > 22 || L < 1 || L > 126) return NULL;
    orc_lit_table *t = (orc_lit_table *)calloc(1, sizeof(*t));
    if (!t) return NULL;
    t->S = S; t->m = m; t->row_bytes = row_bytes; t->R = R; t->L = L; t->a1 = a1; t->a2 = a2;
    t->c = (int32_t *)malloc(sizeof(int32_t) * S);
    t->q = (uint32_t *)malloc(sizeof(uint32_t) * S);
    t->rows = (uint8_t *)calloc((size_t)S, row_bytes ? row_bytes : 1);
    if (!t->c || !t->q || !t->rows) { free(t->c); free(t->q); free(t->rows); free(t); return NULL; }
    for (uint32_t j = 0; j < S; ++j) { t->c[j] = -1; t->q[j] = 0xFF800000u; }   /* dead, invalid mapping */
    return t;
}

void orc_lit_destroy(orc_lit_table *t)
{
    if (!t) return;
    free(t->c); free(t->q); free(t->rows); free(t);
}

/* Eq. 9-11: bounded double-hashing probe.  Returns 1 on a hit; *h_out is the matching bucket on a hit or
 * the last examined bucket on a miss. */
static int lit_probe(const orc_lit_table *t, int32_t x, uint32_t *h_out)
{
    const uint32_t S = t->S;
    uint32_t h = (t->a1 * (uint32_t)x) % S;
    const uint32_t d = ((t->a2 * (uint32_t)x) % S) | 1u;
    int m = 0;
    for (uint32_t r = 0; r <= t->R; ++r) {
        const uint32_t o = t->q[h] % S;
        m = (t->c[o] == x);
        if (m || r == t->R) break;
        h = (h + d) % S;
    }
    *h_out = h;
    return m;
}

/* Eq. 4 with the decode chain of App. F. */
static int lit_reusable(const orc_lit_table *t, uint32_t h)
{
    const uint32_t S = t->S, F = 1u << (23 - t->m);
    const uint32_t u = t->q[h] % (2u * F * S);
    const uint32_t b = u / (F * S), o = u % S, phi_h = (u % (F * S)) / S;
    return b == 1 || lit_life(t->q[o]) < 0 || phi_h != ((uint32_t)t->c[o] % F);
}

static void lit_decay_all(orc_lit_table *t)
{
    for (uint32_t j = 0; j < t->S; ++j) {
        int32_t l = lit_life(t->q[j]);
        if (l > -1) t->q[j] = lit_set_life(t->q[j], l - 1);
    }
}

/* Algorithm 1 with the literal Probe and UpdateState (Algorithm 2). */
int32_t orc_lit_stage_one_token(orc_lit_table *t, uint32_t g, const int32_t *x, uint32_t K,
                                int32_t *o, uint8_t *m, orc_xfer *list, uint32_t *n_list)
{
    const uint32_t S = t->S, F = 1u << (23 - t->m);
    int32_t *e = (int32_t *)malloc(sizeof(int32_t) * S);
    uint32_t *hb = (uint32_t *)malloc(sizeof(uint32_t) * (K ? K : 1));
    uint8_t *vb = (uint8_t *)malloc(K ? K : 1);
    if (!e || !hb || !vb) { free(e); free(hb); free(vb); return ORC_ENOMEM; }

    if (g == 0) lit_decay_all(t);
    for (uint32_t i = 0; i < K; ++i) {                       /* Probe: hit mask m and bucket indices h */
        m[i] = 0; o[i] = -1;
        if (x[i] < 0) continue;
        uint32_t h;
        if (lit_probe(t, x[i], &h)) { m[i] = 1; o[i] = (int32_t)(t->q[h] % S); }
    }
    for (uint32_t i = 0; i < K; ++i)
        if (m[i]) t->q[o[i]] = lit_set_life(t->q[o[i]], t->L);
    int32_t n_g = 0;
    uint32_t valid = 0;
    for (uint32_t i = 0; i < K; ++i)
        if (x[i] >= 0) { valid++; n_g += 1 - (int32_t)m[i]; }

    uint32_t n_dead = 0;
    for (;;) {                                               /* CollectDead / decay loop */
        n_dead = 0;
        for (uint32_t j = 0; j < S; ++j) if (lit_life(t->q[j]) < 0) e[n_dead++] = (int32_t)j;
        if (n_dead >= (uint32_t)n_g) break;
        int any_alive = 0;
        for (uint32_t j = 0; j < S; ++j) any_alive |= lit_life(t->q[j]) >= 0;
        if (!any_alive) { free(e); free(hb); free(vb); return ORC_ECAPACITY; }
        lit_decay_all(t);
        t->extra_decays++;
    }

    /* UpdateState: (1) all probes on the table as it stands */
    uint32_t k = 0;
    for (uint32_t i = 0; i < K; ++i) {
        if (x[i] < 0 || m[i]) continue;
        uint32_t h = (t->a1 * (uint32_t)x[i]) % S;
        const uint32_t d = ((t->a2 * (uint32_t)x[i]) % S) | 1u;
        int v = 0;
        for (uint32_t r = 0; r <= t->R; ++r) {
            v = lit_reusable(t, h);
            if (v || r == t->R) break;
            h = (h + d) % S;
        }
        hb[k] = h; vb[k] = (uint8_t)v; ++k;
    }
    /* (2) every miss writes its id and lifetime into its allocated slot */
    k = 0;
    for (uint32_t i = 0; i < K; ++i) {
        if (x[i] < 0 || m[i]) continue;
        const int32_t j = e[k++];
        t->c[j] = x[i];
        t->q[j] = lit_set_life(t->q[j], t->L);
        o[i] = j;
        list[*n_list].x = x[i]; list[*n_list].o = j; (*n_list)++;
    }
    /* (3) bucket words, in position order: a later miss overwrites an earlier one on the same bucket */
    k = 0;
    for (uint32_t i = 0; i < K; ++i) {
        if (x[i] < 0 || m[i]) continue;
        if (vb[k]) {
            const uint32_t h = hb[k];
            t->q[h] = (t->q[h] & 0xFF000000u) | (((uint32_t)x[i] % F) << t->m) | (uint32_t)o[i];
        } else {
            t->lost_mappings++;
        }
        ++k;
    }
    t->tokens++;
    t->hits += valid - (uint32_t)n_g;
    t->misses += (uint32_t)n_g;
    free(e); free(hb); free(vb);
    return n_g;
}

int orc_lit_step(orc_lit_table *t, const int32_t *X, uint32_t N_q, uint32_t K, int32_t N,
                 const uint8_t *host_kv, uint64_t row_stride,
                 int32_t *O, uint8_t *M, int32_t *n, orc_xfer *list, uint32_t *n_list)
{
    if ((uint64_t)N_q * K > t->S) return ORC_ECAPACITY;
    *n_list = 0;
    for (uint32_t g = 0; g < N_q; ++g) {
        int32_t r = orc_lit_stage_one_token(t, g, X + (size_t)g * K, K, O + (size_t)g * K, M + (size_t)g * K, list, n_list);
        if (r < 0) return r;
        n[g] = r;
    }
    if (host_kv)
        for (uint32_t k = 0; k < *n_list; ++k)
            memcpy(t->rows + (size_t)list[k].o * t->row_bytes, host_kv + (uint64_t)list[k].x * row_stride, t->row_bytes);
    t->rows_copied += *n_list;
    for (uint32_t j = 0; j < t->S; ++j) if (t->c[j] >= N) t->c[j] = -1;
    t->steps++;
    return ORC_OK;
}

void orc_lit_export(const orc_lit_table *t, int32_t *c, uint32_t *q)
{
    memcpy(c, t->c, sizeof(int32_t) * t->S);
    memcpy(q, t->q, sizeof(uint32_t) * t->S);
}
void orc_lit_import(orc_lit_table *t, const int32_t *c, const uint32_t *q)
{
    memcpy(t->c, c, sizeof(int32_t) * t->S);
    memcpy(t->q, q, sizeof(uint32_t) * t->S);
}
const uint8_t *orc_lit_rows(const orc_lit_table *t) { return t->rows; }
void orc_lit_counters(const orc_lit_table *t, uint64_t out[7])
{
    out[0] = t->steps; out[1] = t->tokens; out[2] = t->hits; out[3] = t->misses;
    out[4] = t->rows_copied; out[5] = t->extra_decays; out[6] = t->lost_mappings;
}
