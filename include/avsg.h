/*
 * avsg.h - C ABI of the AVSG per-decode-step operator for NVIDIA B200 (sm_100a).
 *
 * For every request's top-K selected token ids of one decode iteration the
 * operator (paper Sec. 3.1, Algorithm 4)
 *   1. matches the ids against a device-resident KV buffer of S slots
 *      (hit / miss, Eq. 1),
 *   2. reserves slots for the misses under the lifetime policy (Algorithm 1
 *      passes 1-3, Algorithm 3, CollectDead Eq. 12); the tokens of one
 *      multi-token-prediction iteration are processed in order through one
 *      shared table (Sec. 3.6),
 *   3. copies only the missed KV rows from host memory into their slots, the
 *      miss list being cut evenly over all SMs (Sec. 3.4, Eq. 6),
 *   4. forgets speculative entries (ids >= verified length, end of Alg. 4),
 * and returns the slot table that sparse attention reads.
 *
 * Conventions
 *   - "table" = one persistent (request, layer) buffer with its state.
 *   - Every function returns AVSG_OK (0) or a negative AVSG_E* code and never
 *     throws, traps or aborts.  avsg_strerror() names a code.
 *   - Pointers are marked HOST or DEVICE.  The library never takes ownership
 *     of caller memory.  The context owns all state, the KV buffers and the
 *     scratch it needs; everything is allocated in avsg_create().
 *   - Calls on one context must not overlap in time (one stream at a time).
 *     Different contexts share nothing: their calls may run on different
 *     streams, or be issued by different host threads, at the same time.
 *   - Kernel-side problems (a bounded loop that ran out, a slot or segment
 *     index out of range, an id beyond kv_rows or the direct index) never
 *     fault: the kernel records a code in a status word that avsg_stats(),
 *     avsg_export_state() and avsg_sync_status() report as
 *     AVSG_EDEVICE_STATUS.  An id beyond a table's host rows is only caught
 *     when the call states kv_rows: the library cannot know the extent of
 *     the caller's host allocation otherwise.
 */
#ifndef AVSG_H
#define AVSG_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define AVSG_OK              0
#define AVSG_EINVAL         -1   /* bad argument                                        */
#define AVSG_ENOMEM         -2   /* host or device allocation failed                    */
#define AVSG_ECUDA          -3   /* a CUDA runtime call failed                          */
#define AVSG_ECAPACITY      -4   /* buffer_slots < n_tokens * topk (Eq. 7 violated)     */
#define AVSG_EDEVICE_STATUS -5   /* a kernel reported a problem in the status word      */
#define AVSG_EUNSUPPORTED   -6   /* shape outside what this build supports              */

/* Bits of the device status word (avsg_sync_status).  The word is sticky until
 * avsg_clear_status(). */
#define AVSG_STATUS_PROBE_EXHAUSTED 0x01u /* hash index: a probe visited every bucket          */
#define AVSG_STATUS_NO_DEAD_SLOTS   0x02u /* fewer reclaimable slots than misses (Eq. 7)        */
#define AVSG_STATUS_BAD_SLOT        0x04u /* a slot or position index out of range              */
#define AVSG_STATUS_BAD_SEGMENT     0x08u /* Stage Two could not resolve a miss-list entry      */
#define AVSG_STATUS_BAD_ID          0x10u /* an id >= kv_rows of its table, or >= max_context
                                             with the direct index (taken as padding)          */
#define AVSG_STATUS_WAIT_TIMEOUT    0x20u /* overlapped Stage Two gave up waiting for Stage One:
                                             rows of THAT call were not copied.  Later calls are
                                             not affected (the hand-over flags carry the number
                                             of their call)                                     */
#define AVSG_STATUS_LAUNCH_FAILED   0x40u /* a Stage Two launch failed after Stage One had run:
                                             slots were reserved whose rows were never copied  */

/* How Stage Two moves the missed rows (Sec. 3.4; App. D strategies). */
#define AVSG_XFER_SM_BALANCED   0u  /* miss list cut evenly over all SMs (the operator)  */
#define AVSG_XFER_COPY_ENGINE   1u  /* comparator: miss list read back, one async copy
                                       per run of consecutive rows on the copy engine    */
#define AVSG_XFER_REQUEST_LEVEL 2u  /* comparator S1: one thread block per request       */
#define AVSG_XFER_ALL_K         3u  /* comparator "KV offload": no reuse, all n_tokens*K
                                       rows move; position (g,i) -> slot g*K+i           */
#define AVSG_XFER_POSITION_LEVEL 4u /* comparator S2 (Eq. 14): all top-K positions of the
                                       call are cut into equal ranges, one per thread
                                       block, which walks its range and copies the misses;
                                       hit positions are visited for nothing             */
#define AVSG_XFER_SM_OVERLAP    5u  /* the operator with Stage Two overlapping Stage One
                                       (App. G, latency hiding): the transfer kernel is
                                       resident while Stage One runs and starts on token
                                       g's misses, cut evenly over all SMs per token,
                                       while token g+1 is being placed.  Same results.
                                       A call whose Stage One, with a block per table,
                                       would take more than half of the SMs is served in
                                       rounds of 32 tables: Stage One stays on 32 SMs and
                                       the transfer copies round r's misses while round
                                       r + 1 is matched.  Calls with more than 8 tokens
                                       or 1024 tables, and large calls with a thread-
                                       block cluster per table or AVSG_INDEX_PAPER, run
                                       as AVSG_XFER_SM_BALANCED                          */

/* How Stage One finds the slot that holds an id (same results either way). */
#define AVSG_INDEX_HASH   0u  /* open-addressing table in shared memory, rebuilt every step     */
#define AVSG_INDEX_DIRECT 1u  /* one 16-bit entry per context position in device memory
                                 (2 bytes x max_context per table, L2-resident); needs every
                                 id < max_context                                              */
#define AVSG_INDEX_PAPER  2u  /* the paper's Hash-State table as printed (Eq. 2-4, Eq. 8-11,
                                 Alg. 2): packed 64-bit entries, double hashing with a retry
                                 budget, fingerprints, lazy reclamation.  LOSSY: a resident id
                                 whose bucket word was overwritten is missed and fetched again,
                                 so hit rates are lower than with the two exact indexes.  For
                                 studying the paper's table, not for production use.           */

typedef struct avsg_ctx avsg_ctx;   /* opaque */

typedef struct {
    uint32_t num_tables;     /* persistent tables, each with its own S-slot buffer      */
    uint32_t buffer_slots;   /* S: power of two, 32 .. 32768 (AVSG_INDEX_PAPER: .. 8192) */
    uint32_t row_bytes;      /* bytes per KV row, multiple of 16                        */
    uint32_t max_topk;       /* largest K of any step                                   */
    uint32_t max_tokens;     /* largest N_q = N_mtp + 1; max_tokens*max_topk <= S (Eq. 7) */
    int32_t  max_lifetime;   /* L in 1 .. 126 (paper default 16)                        */
    uint32_t transfer_mode;  /* AVSG_XFER_*                                             */
    int32_t  device;         /* CUDA device ordinal                                     */
    uint32_t index_mode;     /* AVSG_INDEX_*                                            */
    uint32_t max_context;    /* AVSG_INDEX_DIRECT: ids are < max_context (count the
                                speculative positions too); ignored otherwise            */
    uint32_t probe_retries;  /* AVSG_INDEX_PAPER: R, buckets per id = R + 1 (0 = the
                                paper's default 3)                                       */
    uint32_t hash_a1;        /* AVSG_INDEX_PAPER: the two distinct odd primes of Eq. 9   */
    uint32_t hash_a2;        /*   (0 = 1000003 and 998244353; the paper names none)      */
    uint32_t stage_one_cluster; /* thread blocks that share one table in Stage One: 0 = chosen by
                                the library (one block while the table fits one SM's shared
                                memory, i.e. S <= 8192; above that the smallest thread-block
                                cluster that holds it), or 1, 2, 4, 8.  Same results.  Not with
                                AVSG_INDEX_PAPER; needs S / cluster >= 32                */
} avsg_config;

typedef struct {
    uint32_t        n;             /* tables taking part in this call (1 .. num_tables,
                                      at most 2048)                                      */
    const uint32_t *table_ids;     /* HOST [n]   distinct, each < num_tables             */
    uint32_t        n_tokens;      /* N_q of this call (<= max_tokens)                   */
    uint32_t        topk;          /* K of this call (<= max_topk)                       */
    const int32_t  *indices;       /* DEVICE [n][n_tokens][topk] selected ids; unique
                                      within a token; negative = padding                 */
    const void *const *kv_base;    /* HOST [n]   per table: base of its host KV, pinned
                                      (cudaHostAlloc / cudaHostRegister) so the GPU can
                                      read it in place; a device pointer also works      */
    const uint64_t *row_stride;    /* HOST [n] bytes between host rows, multiple of 16;
                                      NULL = row_bytes                                   */
    const int32_t  *verified_len;  /* HOST [n]   N of Alg. 4: ids >= N are speculative   */
    int32_t        *slots;         /* DEVICE out [n][n_tokens][topk]: slot per id,
                                      -1 for padding                                     */
    uint8_t        *hit;           /* DEVICE out [n][n_tokens][topk] 1 = hit, or NULL    */
    int32_t        *miss_count;    /* DEVICE out [n][n_tokens] n_g per token, or NULL    */
    const int32_t  *verified_len_dev; /* DEVICE [n] or NULL.  When set it replaces
                                      verified_len (which may then be NULL): the kernel
                                      reads N when it runs, so that a call captured in a
                                      CUDA graph follows a sequence that grows between
                                      replays                                            */
    const uint32_t *kv_rows;       /* HOST [n] or NULL: rows each table's host KV holds.
                                      When given, an id >= kv_rows[i] is never fetched:
                                      it is taken as padding (slot -1) and reported as
                                      AVSG_STATUS_BAD_ID.  Without it ids are not checked
                                      against the host allocation (the direct index still
                                      bounds them by max_context)                        */
    uint64_t       *stage_one_done; /* DEVICE or NULL (latency hiding, App. G / Sec. 6): when
                                      given, the library stores stage_one_done_value there
                                      (8-byte aligned; device-scope release) as soon as
                                      Stage One has finished every table of the call, i.e.
                                      slots, hit and miss_count are final and every row
                                      that was resident BEFORE the call can be read, while
                                      Stage Two is still copying the missed rows.  Those are
                                      all hits of the first token; a hit of a later token
                                      may be on a slot that an earlier token of the same
                                      call has just reserved (Sec. 3.6) - that slot is also
                                      the slot of a missed position of an earlier token of
                                      the table - and its row is still on its way.  A consumer on another
                                      stream waits for the value with a stream wait-value
                                      operation and starts on the hits; it still has to
                                      wait for the call's stream before it reads a missed
                                      row.  Quicker: a consumer kernel launched right behind
                                      avsg_step on the SAME stream with programmatic stream
                                      serialization (the operator's kernels release their
                                      dependents as soon as they run, and all their blocks
                                      are resident by then): it polls the word, works on
                                      the hits, and executes griddepcontrol.wait before it
                                      touches a missed row.  avsg_step only:
                                      avsg_step_host (which returns its outputs that early
                                      by itself) and AVSG_XFER_ALL_K (no hits) refuse it
                                      with AVSG_EINVAL                                   */
    uint64_t        stage_one_done_value; /* what is stored; the caller chooses values that
                                      let it tell calls apart (e.g. a running count).  A
                                      call captured in a CUDA graph stores the value it was
                                      captured with on every replay: reset the word between
                                      replays, or wait for it with a comparison that the
                                      consumer re-arms                                   */
    uint8_t        *arriving;      /* DEVICE out [n][n_tokens][topk] or NULL (Sec. 3.6 with
                                      Sec. 6): 1 where the position's row comes with THIS
                                      call's Stage Two - it missed, or it hit a slot that an
                                      earlier token of the call had just reserved -, 0 where
                                      the row was resident before the call (readable once
                                      stage_one_done is written) and for padding.  Written
                                      before stage_one_done.  avsg_step only, like
                                      stage_one_done                                     */
} avsg_step_args;

typedef struct {
    uint64_t steps;            /* avsg_step calls x tables                               */
    uint64_t tokens;           /* query tokens processed                                 */
    uint64_t hits, misses;     /* over all valid ids                                     */
    uint64_t rows_copied;      /* rows moved host -> device                              */
    uint64_t bytes_copied;     /* rows_copied * row_bytes                                */
    uint64_t extra_decays;     /* unit decays beyond the pre-decay (Alg. 1 while-loop)   */
    float    last_stage_one_us;/* device time of the last call's match+reserve kernels
                                  and of its transfer; 0 unless timing is enabled.  With
                                  AVSG_XFER_SM_OVERLAP no event separates the two grids:
                                  last_stage_one_us then covers the whole call and
                                  last_transfer_us is ~0                                 */
    float    last_transfer_us;
    uint64_t last_rows;        /* rows the last call moved                               */
    float    last_stage_one_kernel_us; /* the same two grids timed from inside: first block's
                                  start to last block's end on the GPU's own clock, i.e.
                                  without the launch gap an event pair includes; 0 unless
                                  timing is enabled                                       */
    float    last_transfer_kernel_us;
    float    last_transfer_start_us;   /* first transfer block's start after the first Stage One
                                  block's start, same clock: below last_stage_one_kernel_us
                                  when AVSG_XFER_SM_OVERLAP overlaps the two                */
    float    last_copy_start_us;       /* more marks of the last timed call, all counted from the
                                  first Stage One block's start on the GPU's clock: the first
                                  transfer block enters its copy loop (what precedes it is the
                                  part of Stage One the call cannot hide),                   */
    float    last_first_row_us;        /* the first row has arrived from host memory,           */
    float    last_first_block_done_us; /* the first transfer block has copied its share (the
                                  tail of the copy starts here),                             */
    float    last_call_kernel_us;      /* the last block of either grid has ended               */
    float    reserved;
} avsg_stats_t;

/* App. E (a request starts with nothing cached), Sec. 3.1-3.2 (one S-slot
 * buffer plus S state entries per request): allocates all state, every table
 * empty (id -1) and dead (lifetime -1), buffers zeroed.  *out is set only on
 * success.  Tables above 8192 slots are handled by a thread-block cluster
 * per table (stage_one_cluster).  Every kernel of the library is loaded here,
 * so that no later call has to wait for the device's other streams (the CUDA
 * runtime loads a kernel when it is first used, and that may wait for every
 * stream - forever, if one of them waits for a call's stage_one_done word). */
int avsg_create(const avsg_config *cfg, avsg_ctx **out);

/* No passage of the paper: releases everything avsg_create allocated, after
 * waiting for the device.  The pointer is dead afterwards. */
int avsg_destroy(avsg_ctx *ctx);

/* App. E: the next request served by a table starts with an empty cache.  The
 * listed tables become empty and dead again, their rows and counters zero.
 * HOST table_ids[n].  Synchronous. */
int avsg_reset(avsg_ctx *ctx, const uint32_t *table_ids, uint32_t n);

/* The same (App. E), stream-ordered: one kernel on cuda_stream, after the
 * calls issued to that stream before it and before those issued after it;
 * nothing waits on the host.  What a serving loop uses when a request leaves
 * the batch. */
int avsg_reset_async(avsg_ctx *ctx, const uint32_t *table_ids, uint32_t n, void *cuda_stream);

/* Algorithm 4 (with Algorithm 1 and 3 per token, Sec. 3.4 for the gather): one
 * decode iteration for the listed tables, asynchronous on
 * cuda_stream (a cudaStream_t; NULL = default stream).  When the stream has
 * finished this call, buffer[table][slots[...]] holds host row x for every
 * non-padding id x.  Host KV, indices and outputs must stay valid until then.
 * Host arrays of the argument block are consumed before the call returns. */
int avsg_step(avsg_ctx *ctx, const avsg_step_args *args, void *cuda_stream);

/* Same operation (Algorithm 4), but indices / slots / hit / miss_count are HOST pointers (pinned for
 * asynchrony); the library stages them through its own device buffers on the
 * stream: one upload of the ids, one download per requested output. */
int avsg_step_host(avsg_ctx *ctx, const avsg_step_args *args, void *cuda_stream);

/* Sec. 3.1: the S-slot device buffer that sparse attention reads through the
 * slot matrix O.  Returns the DEVICE base of a table's S rows of row_bytes. */
int avsg_buffer(avsg_ctx *ctx, uint32_t table_id, void **d_rows);

/* Sec. 4.4 (hit rate) and App. D (effective bandwidth V / t with V = row_bytes
 * x missed rows): waits for the device, then reports the cumulative counters
 * those figures are formed from.  Returns AVSG_EDEVICE_STATUS (and still fills
 * *out) if a kernel flagged a problem. */
int avsg_stats(avsg_ctx *ctx, avsg_stats_t *out);

/* The same counters for ONE table (the last_* fields stay zero): what the
 * request-level hit rates of Sec. 4.4 / App. E are averaged from.  Waits for
 * the device. */
int avsg_table_stats(avsg_ctx *ctx, uint32_t table_id, avsg_stats_t *out);

/* No passage of the paper (error reporting): waits for the device; returns
 * AVSG_EDEVICE_STATUS if a kernel flagged a problem, and the raw status word
 * in *status_word when not NULL. */
int avsg_sync_status(avsg_ctx *ctx, uint32_t *status_word);

/* No passage of the paper: waits for the device and zeroes the status word. */
int avsg_clear_status(avsg_ctx *ctx);

/* Diagnostic for AVSG_XFER_SM_OVERLAP: launches the overlapped transfer kernel
 * alone on cuda_stream, waiting for a Stage One that is never launched.  Its
 * blocks poll up to their limit (about 0.2 s), raise AVSG_STATUS_WAIT_TIMEOUT,
 * copy nothing and return: a lost Stage One cannot hang the stream, and the
 * context stays usable (clear the status word afterwards).  The paper has no
 * counterpart; its Stage Two starts after Stage One (Alg. 4). */
int avsg_probe_wait_limit(avsg_ctx *ctx, void *cuda_stream);

/* Sec. 3.2: the state of a table is its S entries (cached id c_j, lifetime);
 * these two calls read and replace it, for checkpoints and parity checks.
 * HOST tok[S] (cached id per slot, -1 empty) and life[S] (lifetime, -1 dead).
 * Synchronous. */
int avsg_export_state(avsg_ctx *ctx, uint32_t table_id, int32_t *tok, int8_t *life);
int avsg_import_state(avsg_ctx *ctx, uint32_t table_id, const int32_t *tok, const int8_t *life);

/* AVSG_INDEX_PAPER only: the packed words q[S] (Eq. 2) next to the ids c[S] = tok[S].  avsg_import_state
 * in that mode keeps ids and lifetimes but marks every bucket mapping invalid. */
int avsg_export_hash_state(avsg_ctx *ctx, uint32_t table_id, int32_t *c, uint32_t *q);
int avsg_import_hash_state(avsg_ctx *ctx, uint32_t table_id, const int32_t *c, const uint32_t *q);

/* App. C times Stage One as the median over repeated runs of one step: a
 * device-side snapshot of every table's (tok, life) and its restore, both
 * asynchronous on the stream, let a measurement replay one step many times. */
int avsg_save_state(avsg_ctx *ctx, void *cuda_stream);
int avsg_restore_state(avsg_ctx *ctx, void *cuda_stream);

/* App. D compares transfer strategies on the same misses: switches the Stage
 * Two strategy of later calls (AVSG_XFER_*). */
int avsg_set_transfer_mode(avsg_ctx *ctx, uint32_t mode);

/* App. C / App. D report Stage One and Stage Two times separately.  enable
 * != 0: later calls record CUDA events around Stage One and Stage Two;
 * avsg_stats() then reports the last call's device times. */
int avsg_set_timing(avsg_ctx *ctx, int enable);

/* Eq. 6 cuts the miss list over C cores: C = thread blocks (0 = one per SM);
 * threads per block is this build's own knob. */
int avsg_set_transfer_geometry(avsg_ctx *ctx, uint32_t blocks, uint32_t threads);

/*
 * avsg_step_noalloc - the same decode iteration for callers that cannot
 * allocate.  (The paper has no counterpart; this is a deployment aid.)
 *
 * Who needs it: a serving engine that hands all free device memory to its own
 * pool at start-up, so that any later cudaMalloc fails, or a caller on a
 * latency-critical path where an allocation (which may synchronise the whole
 * device) is not acceptable.  There is no context object: the caller owns the
 * table state and passes it in on every call, and the library allocates
 * nothing - no cudaMalloc, cudaFree or allocating library routine is called.
 * The scratch the step needs (miss list, per-table segment descriptors,
 * counters, status word) is a fixed array of about 1 MiB inside the library
 * image; every GPU that loads the library holds it until the process exits.
 *
 * Limits (AVSG_EUNSUPPORTED beyond them): n <= AVSG_NOALLOC_MAX_TABLES,
 * n * n_tokens * topk <= AVSG_NOALLOC_MAX_IDS, buffer_slots <= 8192.
 * buffer_slots < n_tokens * topk returns AVSG_ECAPACITY.
 *
 * Runs on the CURRENT device, asynchronously on cuda_stream.  The first call
 * on a device also looks up the device address of the scratch array and sets
 * the kernel's shared-memory limit; make that first call outside any stream
 * capture.  All calls on a device share the one scratch array: calls that
 * overlap on the GPU (two streams, or two host threads) race on it, so keep
 * them on one stream or order them yourself.  The array keeps the previous
 * call's contents; the library clears what has to start at zero.
 *
 * State layout (caller-owned DEVICE memory, table i at index i):
 *   tok    int32 [n][buffer_slots]  cached id per slot; a new table is all -1
 *   life   int8  [n][buffer_slots]  lifetime per slot;  a new table is all -1
 *   buffer bytes [n][buffer_slots * row_bytes]  the KV rows attention reads
 * Results are the same, bit for bit, as avsg_step on a context in the same
 * state.
 */
#define AVSG_NOALLOC_MAX_TABLES 32u
#define AVSG_NOALLOC_MAX_IDS    131072u   /* n * n_tokens * topk of one call */

typedef struct {
    uint32_t        n;             /* tables in this call                                */
    uint32_t        n_tokens;      /* N_q                                                */
    uint32_t        topk;          /* K                                                  */
    uint32_t        buffer_slots;  /* S: power of two, 32 .. 8192                        */
    uint32_t        row_bytes;     /* multiple of 16                                     */
    int32_t         max_lifetime;  /* L in 1 .. 126                                      */
    int32_t        *tok;           /* DEVICE in/out [n][S]                               */
    int8_t         *life;          /* DEVICE in/out [n][S]                               */
    void           *buffer;        /* DEVICE in/out [n][S * row_bytes]                   */
    const int32_t  *indices;       /* DEVICE [n][n_tokens][topk]                         */
    const void *const *kv_base;    /* HOST [n]: pinned host KV base per table            */
    const uint64_t *row_stride;    /* HOST [n] or NULL (= row_bytes)                     */
    const int32_t  *verified_len;  /* HOST [n]                                           */
    int32_t        *slots;         /* DEVICE out [n][n_tokens][topk]                     */
    uint8_t        *hit;           /* DEVICE out or NULL                                 */
    int32_t        *miss_count;    /* DEVICE out [n][n_tokens] or NULL                   */
    uint32_t       *status;        /* DEVICE out or NULL: 0, or the kernels' status bits */
    const uint32_t *kv_rows;       /* HOST [n] or NULL: rows of each table's host KV; an
                                      id at or beyond it is not fetched (see avsg_step_args) */
} avsg_noalloc_args;

int avsg_step_noalloc(const avsg_noalloc_args *args, void *cuda_stream);

/*
 * App. G (the host KV pool is an mmap of huge pages): page-locked,
 * device-mapped HOST memory for a table's host KV, for callers that do not
 * bring their own pool.  Any pinned, device-mapped memory serves as kv_base;
 * this is one way to get it.
 *
 * The range is an anonymous private mapping aligned to 2 MiB, touched page by
 * page by the CALLING thread (so it lands on that thread's NUMA node: bind the
 * thread first) and registered with the CUDA runtime for the current device's
 * context (portable, mapped).  With AVSG_HOST_KV_HUGE_PAGES the kernel is
 * asked, before the first touch, to back it with transparent 2 MiB pages; the
 * request is advisory, the memory is valid either way.  Contents start as
 * zeros.
 *   bytes        > 0; rounded up to 2 MiB internally
 *   out          HOST: receives the base address (host pointer; usable as
 *                kv_base as it is)
 *   huge_bytes   HOST or NULL: receives how many bytes of the range the kernel
 *                reports as backed by huge pages right after the touch
 *                (0 when it cannot be read)
 * AVSG_EINVAL for bad arguments, AVSG_ENOMEM when the mapping fails,
 * AVSG_ECUDA when registration fails (the mapping is released again).
 *
 * avsg_host_kv_free: unregisters and unmaps a range avsg_host_kv_alloc
 * returned; no call that reads it may be in flight.  AVSG_EINVAL for a pointer
 * that did not come from avsg_host_kv_alloc (or was freed already).
 */
#define AVSG_HOST_KV_HUGE_PAGES 1u
int avsg_host_kv_alloc(size_t bytes, uint32_t flags, void **out, uint64_t *huge_bytes);
int avsg_host_kv_free(void *base);

/* No passage of the paper: a static string naming an AVSG_E* code. */
const char *avsg_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* AVSG_H */
