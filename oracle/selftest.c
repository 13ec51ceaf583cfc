/*
 * Sanitizer self-test of the oracle (test infrastructure): drives both oracle modes over random traces and
 * checks the invariants that need no second implementation.  Built by tests/test_oracle_sanitizers.py with
 * -fsanitize=address,undefined together with avsg_oracle.c; any out-of-bounds access, leak or undefined
 * operation in the oracle aborts the run.
 */
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

typedef struct orc_table orc_table;
typedef struct orc_lit_table orc_lit_table;
typedef struct { int32_t x; int32_t o; } orc_xfer;
orc_table *orc_create(uint32_t S, uint32_t row_bytes, int32_t L);
void orc_destroy(orc_table *t);
int orc_step(orc_table *t, const int32_t *X, uint32_t N_q, uint32_t K, int32_t N, const uint8_t *host_kv,
             uint64_t row_stride, int32_t *O, uint8_t *M, int32_t *n, orc_xfer *list, uint32_t *n_list);
void orc_export(const orc_table *t, int32_t *c, int8_t *life);
orc_lit_table *orc_lit_create(uint32_t S, uint32_t row_bytes, int32_t L, uint32_t R, uint32_t a1, uint32_t a2);
void orc_lit_destroy(orc_lit_table *t);
int orc_lit_step(orc_lit_table *t, const int32_t *X, uint32_t N_q, uint32_t K, int32_t N, const uint8_t *host_kv,
                 uint64_t row_stride, int32_t *O, uint8_t *M, int32_t *n, orc_xfer *list, uint32_t *n_list);
void orc_lit_export(const orc_lit_table *t, int32_t *c, uint32_t *q);

static uint64_t rng_state = 88172645463325252ull;
static uint32_t rnd(void) { rng_state ^= rng_state << 13; rng_state ^= rng_state >> 7; rng_state ^= rng_state << 17; return (uint32_t)(rng_state >> 16); }

static int cmp(const void *a, const void *b) { int32_t x = *(const int32_t *)a, y = *(const int32_t *)b; return (x > y) - (x < y); }

int main(void)
{
    const uint32_t shapes[][4] = {{32, 16, 2, 1}, {64, 16, 4, 3}, {256, 100, 2, 16}, {1024, 256, 1, 16}, {128, 128, 1, 126}};
    for (unsigned s = 0; s < sizeof(shapes) / sizeof(shapes[0]); ++s) {
        const uint32_t S = shapes[s][0], K = shapes[s][1], Nq = shapes[s][2], rb = 48, ctx = 4 * S;
        const int32_t L = (int32_t)shapes[s][3];
        uint8_t *kv = (uint8_t *)malloc((size_t)ctx * rb);
        for (size_t i = 0; i < (size_t)ctx * rb; ++i) kv[i] = (uint8_t)rnd();
        int32_t *X = (int32_t *)malloc(sizeof(int32_t) * Nq * K), *O = (int32_t *)malloc(sizeof(int32_t) * Nq * K);
        uint8_t *M = (uint8_t *)malloc(Nq * K), *mark = (uint8_t *)calloc(ctx, 1);
        int32_t *n = (int32_t *)malloc(sizeof(int32_t) * Nq), *c = (int32_t *)malloc(sizeof(int32_t) * S);
        int8_t *life = (int8_t *)malloc(S);
        uint32_t *q = (uint32_t *)malloc(sizeof(uint32_t) * S);
        orc_xfer *list = (orc_xfer *)malloc(sizeof(orc_xfer) * Nq * K);
        orc_table *t = orc_create(S, rb, L);
        orc_lit_table *lt = orc_lit_create(S, rb, L, 3, 1000003u, 998244353u);
        if (!t || !lt) return 2;
        for (int step = 0; step < 60; ++step) {
            for (uint32_t g = 0; g < Nq; ++g) {          /* K distinct ids per token, some padding now and then */
                uint32_t k = 0;
                memset(mark, 0, ctx);
                while (k < K) { uint32_t id = rnd() % (step % 3 ? ctx / 4 : ctx); if (!mark[id]) { mark[id] = 1; X[g * K + k++] = (int32_t)id; } }
                qsort(X + g * K, K, sizeof(int32_t), cmp);
                if (step % 11 == 10) X[g * K + K - 1] = -1;
            }
            uint32_t nl = 0;
            if (orc_step(t, X, Nq, K, (int32_t)ctx - 3, kv, rb, O, M, n, list, &nl)) return 3;
            orc_export(t, c, life);
            for (uint32_t p = 0; p < Nq * K; ++p) {
                if (X[p] < 0) { if (O[p] != -1) return 4; continue; }
                if (O[p] < 0 || (uint32_t)O[p] >= S) return 5;
                if (X[p] < (int32_t)ctx - 3 && c[O[p]] != X[p]) return 6;
            }
            for (uint32_t j = 0; j < S; ++j) if (life[j] < -1 || life[j] > L || c[j] >= (int32_t)ctx - 3) return 7;
            if (orc_lit_step(lt, X, Nq, K, (int32_t)ctx - 3, kv, rb, O, M, n, list, &nl)) return 8;
            orc_lit_export(lt, c, q);
            for (uint32_t p = 0; p < Nq * K; ++p)
                if (X[p] >= 0 && (O[p] < 0 || (uint32_t)O[p] >= S)) return 9;
        }
        orc_destroy(t); orc_lit_destroy(lt);
        free(kv); free(X); free(O); free(M); free(mark); free(n); free(c); free(life); free(q); free(list);
    }
    printf("oracle selftest ok\n");
    return 0;
}
