/* Host-side driver of the C ABI's argument paths (no GPU needed): every call here is refused before any CUDA
 * work, or fails at the first CUDA call when there is no device.  Built with -fsanitize=address,undefined
 * against a library whose host code is instrumented the same way, it shows that the argument checks read no
 * memory they should not.  Also prints the layout of the public structs for the binding's layout test. */
#include <stddef.h>
#include <stdio.h>
#include <string.h>

#include "avsg.h"

static int failures = 0;
#define EXPECT(call, want) do { int rc_ = (call); if (rc_ != (want)) { \
    printf("FAIL %s -> %d, expected %d\n", #call, rc_, (want)); ++failures; } } while (0)

int main(void)
{
    printf("sizeof avsg_config %zu\n", sizeof(avsg_config));
    printf("sizeof avsg_step_args %zu\n", sizeof(avsg_step_args));
    printf("sizeof avsg_stats_t %zu\n", sizeof(avsg_stats_t));
    printf("sizeof avsg_noalloc_args %zu\n", sizeof(avsg_noalloc_args));
    printf("offsetof avsg_config.stage_one_cluster %zu\n", offsetof(avsg_config, stage_one_cluster));
    printf("offsetof avsg_step_args.kv_rows %zu\n", offsetof(avsg_step_args, kv_rows));
    printf("offsetof avsg_step_args.indices %zu\n", offsetof(avsg_step_args, indices));
    printf("offsetof avsg_noalloc_args.kv_rows %zu\n", offsetof(avsg_noalloc_args, kv_rows));
    printf("offsetof avsg_stats_t.last_rows %zu\n", offsetof(avsg_stats_t, last_rows));

    avsg_ctx *ctx = NULL;
    avsg_config c;
    memset(&c, 0, sizeof(c));
    EXPECT(avsg_create(NULL, &ctx), AVSG_EINVAL);
    EXPECT(avsg_create(&c, NULL), AVSG_EINVAL);
    c.num_tables = 1; c.buffer_slots = 1000; c.row_bytes = 656; c.max_topk = 16; c.max_tokens = 1; c.max_lifetime = 16;
    EXPECT(avsg_create(&c, &ctx), AVSG_EINVAL);                  /* slots not a power of two */
    c.buffer_slots = 16;
    EXPECT(avsg_create(&c, &ctx), AVSG_EINVAL);                  /* fewer than 32 slots */
    c.buffer_slots = 65536;
    EXPECT(avsg_create(&c, &ctx), AVSG_EUNSUPPORTED);
    c.buffer_slots = 1024; c.row_bytes = 650;
    EXPECT(avsg_create(&c, &ctx), AVSG_EINVAL);
    c.row_bytes = 656; c.max_topk = 600; c.max_tokens = 2;
    EXPECT(avsg_create(&c, &ctx), AVSG_ECAPACITY);               /* Eq. 7 */
    c.max_topk = 16; c.max_tokens = 1; c.max_lifetime = 127;
    EXPECT(avsg_create(&c, &ctx), AVSG_EINVAL);
    c.max_lifetime = 16; c.transfer_mode = 6;
    EXPECT(avsg_create(&c, &ctx), AVSG_EINVAL);
    c.transfer_mode = 0; c.index_mode = AVSG_INDEX_DIRECT; c.max_context = 0;
    EXPECT(avsg_create(&c, &ctx), AVSG_EINVAL);
    c.index_mode = 0; c.stage_one_cluster = 3;
    EXPECT(avsg_create(&c, &ctx), AVSG_EINVAL);
    c.stage_one_cluster = 16;
    EXPECT(avsg_create(&c, &ctx), AVSG_EINVAL);
    c.stage_one_cluster = 0; c.device = -1;
    EXPECT(avsg_create(&c, &ctx), AVSG_ECUDA);                   /* no such device (or no device at all) */
    if (ctx != NULL) { printf("FAIL a refused create set *out\n"); ++failures; }

    avsg_stats_t st;
    uint32_t word = 0, ids[2] = {0, 1};
    void *rows = NULL;
    int32_t tok[4]; int8_t life[4]; uint32_t q[4];
    EXPECT(avsg_destroy(NULL), AVSG_EINVAL);
    EXPECT(avsg_reset(NULL, ids, 2), AVSG_EINVAL);
    EXPECT(avsg_reset_async(NULL, ids, 2, NULL), AVSG_EINVAL);
    EXPECT(avsg_step(NULL, NULL, NULL), AVSG_EINVAL);
    EXPECT(avsg_step_host(NULL, NULL, NULL), AVSG_EINVAL);
    EXPECT(avsg_buffer(NULL, 0, &rows), AVSG_EINVAL);
    EXPECT(avsg_stats(NULL, &st), AVSG_EINVAL);
    EXPECT(avsg_table_stats(NULL, 0, &st), AVSG_EINVAL);
    EXPECT(avsg_sync_status(NULL, &word), AVSG_EINVAL);
    EXPECT(avsg_clear_status(NULL), AVSG_EINVAL);
    EXPECT(avsg_probe_wait_limit(NULL, NULL), AVSG_EINVAL);
    EXPECT(avsg_export_state(NULL, 0, tok, life), AVSG_EINVAL);
    EXPECT(avsg_import_state(NULL, 0, tok, life), AVSG_EINVAL);
    EXPECT(avsg_export_hash_state(NULL, 0, tok, q), AVSG_EINVAL);
    EXPECT(avsg_import_hash_state(NULL, 0, tok, q), AVSG_EINVAL);
    EXPECT(avsg_save_state(NULL, NULL), AVSG_EINVAL);
    EXPECT(avsg_restore_state(NULL, NULL), AVSG_EINVAL);
    EXPECT(avsg_set_transfer_mode(NULL, 0), AVSG_EINVAL);
    EXPECT(avsg_set_timing(NULL, 1), AVSG_EINVAL);
    EXPECT(avsg_set_transfer_geometry(NULL, 148, 256), AVSG_EINVAL);

    /* the entry point without a context: sizes are refused before any pointer is touched */
    avsg_noalloc_args a;
    memset(&a, 0, sizeof(a));
    EXPECT(avsg_step_noalloc(NULL, NULL), AVSG_EINVAL);
    EXPECT(avsg_step_noalloc(&a, NULL), AVSG_EINVAL);
    a.n = 1; a.n_tokens = 1; a.topk = 16; a.buffer_slots = 100; a.row_bytes = 32; a.max_lifetime = 16;
    EXPECT(avsg_step_noalloc(&a, NULL), AVSG_EINVAL);            /* slots not a power of two */
    a.buffer_slots = 64;
    EXPECT(avsg_step_noalloc(&a, NULL), AVSG_EINVAL);            /* null state pointers */
    int dummy[4] = {0, 0, 0, 0};
    const void *kv[1] = {dummy};
    int32_t vlen[1] = {4};
    a.tok = dummy; a.life = (int8_t *)dummy; a.buffer = dummy; a.indices = dummy; a.slots = dummy;
    a.kv_base = kv; a.verified_len = vlen;
    a.n = AVSG_NOALLOC_MAX_TABLES + 1;
    EXPECT(avsg_step_noalloc(&a, NULL), AVSG_EUNSUPPORTED);
    a.n = 1; a.buffer_slots = 16384;
    EXPECT(avsg_step_noalloc(&a, NULL), AVSG_EUNSUPPORTED);
    a.buffer_slots = 64; a.n_tokens = 2; a.topk = 40;
    EXPECT(avsg_step_noalloc(&a, NULL), AVSG_ECAPACITY);

    for (int code = 1; code >= -8; --code)
        if (!avsg_strerror(code) || !avsg_strerror(code)[0]) { printf("FAIL no text for code %d\n", code); ++failures; }
    printf("failures %d\n", failures);
    return failures != 0;
}
