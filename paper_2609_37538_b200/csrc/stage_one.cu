// Stage One of the AVSG operator: match + reserve, one thread block per table.
//
// Follows Algorithm 1 (refresh / classify / allocate) with the lifetime
// operations of Algorithm 3, for the N_q tokens of one iteration in order
// (Algorithm 4), and the end-of-step invalidation of Algorithm 4.
//
// Two interchangeable id -> slot indexes (template parameter DIRECT):
//   hash   (default) an open-addressing table in shared memory, rebuilt every step (described below);
//   direct           one 16-bit slot number per context position in global memory (it stays L2-resident:
//                    2 bytes x context per table).  An entry is only ever written when an id is installed
//                    and is never cleared: a lookup masks it to a valid slot number and then compares the
//                    slot's cached id, so stale or uninitialised entries simply miss.  No build, no probing.
//
// The whole table lives in shared memory for the step:
//   s_tok[S]   cached id per slot            s_life[S]  lifetime per slot
//   s_key[H], s_val[H]  open-addressing index id -> slot, H = 2S buckets,
//                       rebuilt from s_tok at the start of every step
// The index is private to this kernel (it is not part of the table state): a
// hit is "some slot holds the id" (Eq. 1), whatever bucket found it.  Entries
// are never deleted: when a slot is reclaimed its old key stays behind and is
// recognised as stale because s_tok[slot] no longer equals the key; a later
// insert of the same id re-uses that bucket, so a key occupies one bucket at
// most.  The index is rebuilt when stale keys would push the load above 3/4.
//
// The decay loop of Algorithm 1 ("decay all, CollectDead, until enough slots
// are dead") is evaluated in closed form: d = the smallest number of unit
// decays after which at least n_g lifetimes are negative, read off a
// histogram of the S lifetimes; the lifetimes then drop by d at once,
// saturating at -1.  For L <= 30 the histogram is counted without atomics:
// every thread bumps private byte counters (one column per thread, one row
// per lifetime value) and one warp per value sums its row with dp4a.  Dead slots are compacted in increasing slot order and
// the k-th miss in position order takes the k-th of them (ballot-free packed
// byte arithmetic + warp/block prefix sums, no atomics, so the assignment is
// deterministic).
//
// When Stage Two overlaps Stage One (S1Params::ready set), the block announces
// every token as soon as its misses are placed: see publish_token().
#include "avsg_kernels.cuh"
#include "stage_one_common.cuh"

namespace avsg {
namespace {

struct Index {
    int32_t*  key;
    uint16_t* val;
    const int32_t* tok;
    uint32_t mask, logH;
};

// Returns the slot holding x, or -1.  Bounded by the number of buckets.
__device__ __forceinline__ int32_t index_find(const Index& ix, int32_t x, uint32_t* status)
{
    uint32_t b = hash_id(x, ix.logH);
    for (uint32_t it = 0; it <= ix.mask; ++it) {
        const int32_t k = ix.key[b];
        if (k == x) {
            const uint32_t j = ix.val[b];
            return ix.tok[j] == x ? (int32_t)j : -1;     // a stale key means the id was reclaimed this step
        }
        if (k == EMPTY) return -1;
        b = (b + 1u) & ix.mask;
    }
    atomicOr(status, ST_PROBE_EXHAUSTED);
    return -1;
}

// Installs x -> slot; re-uses the bucket that already carries x if there is one.
__device__ __forceinline__ void index_insert(const Index& ix, int32_t x, uint32_t slot, uint32_t* status)
{
    uint32_t b = hash_id(x, ix.logH);
    for (uint32_t it = 0; it <= ix.mask; ++it) {
        const int32_t old = atomicCAS(&ix.key[b], EMPTY, x);
        if (old == EMPTY || old == x) { ix.val[b] = (uint16_t)slot; return; }
        b = (b + 1u) & ix.mask;
    }
    atomicOr(status, ST_PROBE_EXHAUSTED);
}

// Inserts the ids of the slots a thread owns.  The first compare-and-swap of every id is issued
// before any result is inspected, so that a thread keeps up to eight shared-memory atomics in flight.
__device__ __forceinline__ void build_index(const Index& ix, const int32_t* s_tok, uint32_t j0, uint32_t spt, bool own,
                                            uint32_t* s_fill, uint32_t* status)
{
    uint32_t live = 0;
    int32_t x[MAX_SPT], old[MAX_SPT];
    uint32_t b[MAX_SPT];
#pragma unroll
    for (uint32_t k = 0; k < (uint32_t)MAX_SPT; ++k) {
        x[k] = (own && k < spt) ? s_tok[j0 + k] : -1;
        if (x[k] >= 0) {
            b[k] = hash_id(x[k], ix.logH);
            old[k] = atomicCAS(&ix.key[b[k]], EMPTY, x[k]);
            ++live;
        }
    }
#pragma unroll
    for (uint32_t k = 0; k < (uint32_t)MAX_SPT; ++k) {
        if (x[k] >= 0) {
            if (old[k] == EMPTY || old[k] == x[k]) {
                ix.val[b[k]] = (uint16_t)(j0 + k);
            } else {
                uint32_t bb = (b[k] + 1u) & ix.mask;
                bool done = false;
                for (uint32_t it = 0; it < ix.mask; ++it) {
                    const int32_t o = atomicCAS(&ix.key[bb], EMPTY, x[k]);
                    if (o == EMPTY || o == x[k]) { ix.val[bb] = (uint16_t)(j0 + k); done = true; break; }
                    bb = (bb + 1u) & ix.mask;
                }
                if (!done) atomicOr(status, ST_PROBE_EXHAUSTED);
            }
        }
    }
    live = __reduce_add_sync(0xffffffffu, live);
    if ((threadIdx.x & 31u) == 0 && live) atomicAdd(s_fill, live);
}

template <bool DIRECT, int CAP, bool ROUNDS>
__global__ void __launch_bounds__(1024, 1) avsg_stage_one_kernel(const __grid_constant__ S1ParamsT<CAP> p)
{
    extern __shared__ __align__(16) unsigned char smem[];
    const uint32_t S = p.S, K = p.K, H = DIRECT ? 0u : 1u << p.logH, Kp = (K + 7u) & ~7u;
    const uint32_t tid = threadIdx.x, nt = blockDim.x;
    const int32_t L = (int32_t)p.L;

    int32_t*  s_tok      = reinterpret_cast<int32_t*>(smem);
    int32_t*  s_key      = s_tok + S;
    int32_t*  s_miss_x   = s_key + H;
    uint16_t* s_val      = reinterpret_cast<uint16_t*>(s_miss_x + Kp);
    uint16_t* s_miss_pos = s_val + H;
    uint16_t* s_dead     = s_miss_pos + Kp;
    int8_t*   s_life     = reinterpret_cast<int8_t*>(s_dead + Kp);
    uint32_t* s_hist     = reinterpret_cast<uint32_t*>(s_life + S);
    uint32_t* s_scan_a   = s_hist + 128;
    uint32_t* s_scan_b   = s_scan_a + 40;
    uint32_t* s_fill     = s_scan_b + 40;
    const uint32_t priv_stride = nt + 4u;                 // +4: rows start in different banks
    uint8_t*  s_priv     = L <= PRIV_HIST_MAX_L ? reinterpret_cast<uint8_t*>(s_fill + 8) : nullptr;

    // Programmatic dependent launch: this grid may have been started while the previous kernel of the stream
    // was still running; nothing is read before that kernel has completed.  The next kernel (Stage Two) is
    // allowed to start its own prologue right away - it waits the same way before it reads the miss list.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (p.t_range && threadIdx.x == 0) atomicMin(p.t_range, global_ns());
    const uint32_t epoch = p.flags ? __ldcg(p.epoch) : 0u;      // the number of this overlapped call

    // The grid usually has one block per table (ROUNDS = false: one pass, bt = blockIdx.x).  A call with many tables
    // and an overlapped Stage Two is launched with fewer blocks than tables (ROUNDS = true): a block then serves the
    // tables bt = blockIdx.x, blockIdx.x + gridDim.x, ... one after the other, so that Stage One stays on a few SMs
    // and publishes its tables round by round while the transfer grid, resident on the other SMs, already copies
    // the earlier rounds' misses.
    auto one_table = [&](const uint32_t bt) {
        const uint32_t ti = p.first + bt;            // table index within the call
        const uint32_t table = p.table_id[bt];
        int32_t* g_tok = p.tok + (size_t)table * S;
        int8_t*  g_life = p.life + (size_t)table * S;

        const uint32_t spt = S >= nt ? S / nt : 1u;           // slots per thread, power of two <= 8
        const uint32_t j0 = tid * spt;
        const bool own = j0 < S;
        const uint32_t ipt = (K + nt - 1) / nt;               // ids per thread, <= 8
        const uint32_t i0 = tid * ipt;

        Index ix{s_key, s_val, s_tok, H - 1u, p.logH};
        uint16_t* where = DIRECT ? p.where + (size_t)table * p.max_context : nullptr;

        // ---- issue every global load first: table state and the first token's ids ----
        int4 t4[MAX_SPT / 4];
        int32_t t1[3];
        uint32_t lw0, lw1;
        if (own) {
            if ((spt & 3u) == 0) {
    #pragma unroll
                for (uint32_t q = 0; q < (uint32_t)MAX_SPT / 4; ++q)
                    if (q < spt / 4) t4[q] = __ldg(reinterpret_cast<const int4*>(g_tok + j0) + q);
            } else {
    #pragma unroll
                for (uint32_t k = 0; k < 3; ++k)
                    if (k < spt) t1[k] = __ldg(g_tok + j0 + k);
            }
        }
        life_load(g_life, j0, spt, own, lw0, lw1);
        int32_t xs[MAX_IPT];
        load_ids(p.indices + (size_t)ti * p.n_q * K, i0, ipt, K, xs);
        const uint32_t id_limit = p.id_limit[bt];

        if constexpr (!DIRECT) {
            for (uint32_t i = tid; i < H / 4; i += nt)
                reinterpret_cast<int4*>(s_key)[i] = make_int4(EMPTY, EMPTY, EMPTY, EMPTY);
        }
        if (s_priv)
            for (uint32_t i = tid; i < ((uint32_t)(L + 2) * priv_stride + 15u) / 16u; i += nt)
                reinterpret_cast<int4*>(s_priv)[i] = make_int4(0, 0, 0, 0);
        if (tid == 0) *s_fill = 0;
        if (own) {
            if ((spt & 3u) == 0) {
    #pragma unroll
                for (uint32_t q = 0; q < (uint32_t)MAX_SPT / 4; ++q)
                    if (q < spt / 4) reinterpret_cast<int4*>(s_tok + j0)[q] = t4[q];
            } else {
    #pragma unroll
                for (uint32_t k = 0; k < 3; ++k)
                    if (k < spt) s_tok[j0 + k] = t1[k];
            }
        }
        // global pre-decay of the iteration's first token (Alg. 1 Pass 1)
        life_store(s_life, j0, spt, own, decay4(lw0, 1), decay4(lw1, 1));
        __syncthreads();
        uint32_t fill_bound = 0;                              // hash index: non-empty buckets (upper bound)
        if (!DIRECT) {
            build_index(ix, s_tok, j0, spt, own, s_fill, p.status);
            __syncthreads();
            fill_bound = *s_fill;
        }

        uint32_t list_off = 0, sum_valid = 0, sum_miss = 0, sum_decay = 0;
        int2* list = p.miss_list + (size_t)ti * p.list_stride;


        for (uint32_t g = 0; g < p.n_q; ++g) {
            const size_t row = ((size_t)ti * p.n_q + g) * K;
            int32_t* O = p.slots + row;
            uint8_t* Hm = p.hit ? p.hit + row : nullptr;
            if (tid < 128) s_hist[tid] = 0;

            // ---- Probe, refresh hits to L, emit hit slots (Pass 1 + Pass 2) ----
            uint32_t missmask = 0, nmiss = 0, nvalid = 0;
            uint32_t cand[MAX_IPT];                             // direct index: candidate slot per id
            check_ids(xs, i0, ipt, K, id_limit, p.status);      // out-of-range ids become padding (id_limit <= max_context)
            if (DIRECT) {
    #pragma unroll
                for (uint32_t k = 0; k < (uint32_t)MAX_IPT; ++k) {   // all loads are issued before any is used
                    cand[k] = 0xFFFFFFFFu;
                    if (k < ipt && i0 + k < K && xs[k] >= 0) cand[k] = __ldcg(where + xs[k]) & (S - 1u);
                }
            }
    #pragma unroll
            for (uint32_t k = 0; k < (uint32_t)MAX_IPT; ++k) {
                const uint32_t i = i0 + k;
                if (k < ipt && i < K) {
                    const int32_t x = xs[k];
                    if (x >= 0 && (!DIRECT || cand[k] != 0xFFFFFFFFu)) {
                        ++nvalid;
                        int32_t j;
                        if (DIRECT) j = s_tok[cand[k]] == x ? (int32_t)cand[k] : -1;
                        else j = index_find(ix, x, p.status);
                        if (j >= 0) {
                            s_life[j] = (int8_t)L;
                            O[i] = j;
                            if (Hm) Hm[i] = 1;
                        } else {
                            missmask |= 1u << k;
                            ++nmiss;
                        }
                    } else {
                        O[i] = -1;
                        if (Hm) Hm[i] = 0;
                    }
                }
            }
            // order-preserving compaction of the misses: t = x[not m]
            uint32_t total;
            uint32_t off = block_excl_scan(nmiss | (nvalid << 16), s_scan_a, total) & 0xFFFFu;
            const uint32_t n_g = total & 0xFFFFu;
            sum_valid += total >> 16;
            sum_miss += n_g;
    #pragma unroll
            for (uint32_t k = 0; k < (uint32_t)MAX_IPT; ++k) {
                if (missmask & (1u << k)) {
                    s_miss_x[off] = xs[k];
                    s_miss_pos[off] = (uint16_t)(i0 + k);
                    ++off;
                }
            }
            // the next token's ids travel while this token's misses are placed
            if (g + 1 < p.n_q) load_ids(p.indices + row + K, i0, ipt, K, xs);
            if (tid == 0 && p.miss_count) p.miss_count[(size_t)ti * p.n_q + g] = (int32_t)n_g;
            if (n_g == 0) { __syncthreads(); publish_token(p, ti, table, g, 0, bt, epoch); continue; }
            __syncthreads();

            // ---- Pass 3: CollectDead; if fewer than n_g slots are dead, decay until enough are ----
            uint32_t w0, w1;
            life_load(s_life, j0, spt, own, w0, w1);
            uint32_t sg0 = w0 & 0x80808080u, sg1 = w1 & 0x80808080u;       // sign bits = dead slots
            uint32_t dtotal, d = 0;
            uint32_t doff = block_excl_scan(__popc(sg0) + __popc(sg1), s_scan_b, dtotal);
            if (dtotal < n_g) {
                // the while-loop of Alg. 1 in closed form: d = fewest unit decays after which n_g slots are dead,
                // read off the histogram of the lifetimes (only needed on this, the rarer, path)
                count_lifetimes(w0, w1, spt, own, L, s_priv, priv_stride, s_hist);
                __syncthreads();
                uint32_t cum = 0;
                bool found = false;
                d = (uint32_t)L + 1u;
                for (uint32_t b = 0; b <= (uint32_t)L + 1u; ++b) {   // bin b counts lifetime b-1; dead after b decays
                    cum += s_hist[b];
                    if (cum >= n_g) { d = b; found = true; break; }
                }
                if (!found && tid == 0) atomicOr(p.status, ST_NO_DEAD_SLOTS);
                w0 = decay4(w0, d);
                w1 = decay4(w1, d);
                life_store(s_life, j0, spt, own, w0, w1);
                sg0 = w0 & 0x80808080u; sg1 = w1 & 0x80808080u;
                doff = block_excl_scan(__popc(sg0) + __popc(sg1), s_scan_b, dtotal);
            }
            // dead slots in increasing order; the first n_g are handed out
    #pragma unroll
            for (uint32_t k = 0; k < (uint32_t)MAX_SPT; ++k) {
                const uint32_t bit = k < 4 ? (sg0 >> (8 * k + 7)) & 1u : (sg1 >> (8 * (k - 4) + 7)) & 1u;
                if (bit) {
                    if (doff < n_g) s_dead[doff] = (uint16_t)(j0 + k);
                    ++doff;
                }
            }
            __syncthreads();

            // ---- install the misses: k-th miss takes the k-th dead slot ----
            const bool rebuild = !DIRECT && fill_bound + n_g > (H / 4u) * 3u;
            const uint32_t n_take = n_g < dtotal ? n_g : dtotal;
            for (uint32_t k = tid; k < n_take; k += nt) {
                const uint32_t j = s_dead[k];
                const int32_t x = s_miss_x[k];
                const uint32_t i = s_miss_pos[k];
                if (j < S && i < K) {
                    s_tok[j] = x;
                    s_life[j] = (int8_t)L;
                    O[i] = (int32_t)j;
                    if (Hm) Hm[i] = 0;
                    list[list_off + k] = make_int2(x, (int32_t)j);
                    if (DIRECT) __stcg(where + x, (uint16_t)j);
                    else if (!rebuild) index_insert(ix, x, j, p.status);
                } else {
                    list[list_off + k] = make_int2(-1, -1);          // Stage Two skips it
                    atomicOr(p.status, ST_BAD_SLOT);
                }
            }
            list_off += n_take;
            sum_decay += d;
            if (!rebuild) {
                fill_bound += n_g;
                __syncthreads();
            } else if constexpr (!DIRECT) {
                __syncthreads();
                for (uint32_t i = tid; i < H / 4; i += nt)
                    reinterpret_cast<int4*>(s_key)[i] = make_int4(EMPTY, EMPTY, EMPTY, EMPTY);
                if (tid == 0) *s_fill = 0;
                __syncthreads();
                build_index(ix, s_tok, j0, spt, own, s_fill, p.status);
                __syncthreads();
                fill_bound = *s_fill;
            }
            publish_token(p, ti, table, g, n_take, bt, epoch);
        }

        // ---- write the table back; speculative entries (id >= N) become empty (Alg. 4) ----
        const int32_t N = p.verified_len_dev ? __ldg(p.verified_len_dev + ti) : p.verified_len[bt];
        if (own) {
            if ((spt & 3u) == 0) {
                for (uint32_t q = 0; q < spt / 4; ++q) {
                    int4 v = reinterpret_cast<const int4*>(s_tok + j0)[q];
                    v.x = v.x >= N ? -1 : v.x; v.y = v.y >= N ? -1 : v.y;
                    v.z = v.z >= N ? -1 : v.z; v.w = v.w >= N ? -1 : v.w;
                    reinterpret_cast<int4*>(g_tok + j0)[q] = v;
                }
            } else {
                for (uint32_t k = 0; k < spt; ++k) {
                    const int32_t v = s_tok[j0 + k];
                    g_tok[j0 + k] = v >= N ? -1 : v;
                }
            }
            uint32_t w0, w1;
            life_load(s_life, j0, spt, own, w0, w1);
            life_store(g_life, j0, spt, own, w0, w1);
        }
        if (tid == 0) {
            SegDesc sd;
            sd.src_base = p.kv_base[bt];
            sd.src_stride = p.kv_stride[bt];
            sd.dst_base = reinterpret_cast<uint64_t>(p.buffer + (size_t)table * S * p.row_bytes);
            sd.count = list_off;
            sd.pad = 0;
            p.seg[ti] = sd;
            TableStats* st = p.stats + table;
            st->steps += 1;
            st->tokens += p.n_q;
            st->hits += sum_valid - sum_miss;
            st->misses += sum_miss;
            st->rows += list_off;
            st->extra_decays += sum_decay;
        }
    };
    if constexpr (ROUNDS) {
        for (uint32_t bt = blockIdx.x; bt < p.n_launch; bt += gridDim.x) {
            if (bt != blockIdx.x) __syncthreads();        // the previous table's last reads of shared memory are over
            one_table(bt);
        }
    } else {
        one_table(blockIdx.x);
    }
    if (p.t_range) {
        __syncthreads();
        if (tid == 0) atomicMax(p.t_range + 1, global_ns());
    }
}

// Direct index: points every resident id at its slot again, after the table state was replaced from outside
// (import, restore of a snapshot).  One thread per slot; ids are unique within a table.
__global__ void avsg_direct_index_from_state_kernel(const int32_t* __restrict__ tok, uint16_t* where,
                                                    uint32_t first_table, uint32_t n_tables, uint32_t S,
                                                    uint32_t max_context)
{
    const size_t n = (size_t)n_tables * S;
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        const uint32_t t = first_table + (uint32_t)(i / S), j = (uint32_t)(i % S);
        const int32_t x = tok[(size_t)t * S + j];
        if (x >= 0 && (uint32_t)x < max_context) where[(size_t)t * max_context + x] = (uint16_t)j;
    }
}


// A request ended: its tables become empty (id -1) and dead (lifetime -1) again, their counters and rows zero;
// in the paper-literal mode every bucket word returns to (lifetime -1, invalid, fingerprint 0, slot 0).  The
// direct index needs no reset: its entries are verified against the cached ids.  Grid (blocks per table, tables).
__global__ void avsg_reset_tables_kernel(const __grid_constant__ ResetParams p)
{
    const uint32_t table = p.table_id[blockIdx.y];
    const size_t S = p.S, tid = blockIdx.x * (size_t)blockDim.x + threadIdx.x, nth = (size_t)gridDim.x * blockDim.x;
    for (size_t j = tid; j < S; j += nth) {
        p.tok[table * S + j] = -1;
        p.life[table * S + j] = (int8_t)-1;
        if (p.qword) p.qword[table * S + j] = 0xFF800000u;
    }
    int4* rows = reinterpret_cast<int4*>(p.buffer + table * S * p.row_bytes);
    for (size_t i = tid; i < S * (p.row_bytes >> 4); i += nth) rows[i] = make_int4(0, 0, 0, 0);
    if (tid == 0) p.stats[table] = TableStats{0, 0, 0, 0, 0, 0};
}

// ---------------------------------------------------------------------------------------------------------------
// Paper-literal Hash-State mode (Sec. 3.2-3.3, Eq. 2-4, Eq. 8-11, Algorithm 2): 64-bit entries (c_j, q_j) with
// q_j = [lifetime 8 | invalid 1 | fingerprint 23-m | slot m], double hashing with retry budget R, fingerprint
// check and lazy reclamation of stale bucket words.  Lossy by design: a resident id whose bucket word was
// overwritten is missed and fetched again.  Where Algorithm 2 leaves open which of several writers of one bucket
// wins, the miss with the highest position wins (an atomicMax on a per-bucket tag), so results are reproducible.
// ---------------------------------------------------------------------------------------------------------------
__device__ __forceinline__ void pack_life_bytes(const uint32_t* q, uint32_t j0, uint32_t spt, bool own,
                                                uint32_t& w0, uint32_t& w1)
{
    w0 = w1 = 0x7F7F7F7Fu;
    if (!own) return;
#pragma unroll
    for (uint32_t k = 0; k < (uint32_t)MAX_SPT; ++k) {
        if (k < spt) {
            const uint32_t b = q[j0 + k] >> 24;
            if (k < 4) w0 = (w0 & ~(0xFFu << (8 * k))) | (b << (8 * k));
            else w1 = (w1 & ~(0xFFu << (8 * (k - 4)))) | (b << (8 * (k - 4)));
        }
    }
}

__device__ __forceinline__ void unpack_life_bytes(uint32_t* q, uint32_t j0, uint32_t spt, bool own, uint32_t w0, uint32_t w1)
{
    if (!own) return;
#pragma unroll
    for (uint32_t k = 0; k < (uint32_t)MAX_SPT; ++k) {
        if (k < spt) {
            const uint32_t b = k < 4 ? (w0 >> (8 * k)) & 0xFFu : (w1 >> (8 * (k - 4))) & 0xFFu;
            q[j0 + k] = (q[j0 + k] & 0x00FFFFFFu) | (b << 24);
        }
    }
}

__global__ void __launch_bounds__(1024, 1) avsg_stage_one_paper_kernel(const __grid_constant__ S1Params p)
{
    extern __shared__ __align__(16) unsigned char smem[];
    const uint32_t S = p.S, K = p.K, Kp = (K + 7u) & ~7u, m = p.logH - 1u, Fm = (1u << (23u - m)) - 1u;
    const uint32_t tid = threadIdx.x, nt = blockDim.x, R = p.probe_retries, a1 = p.hash_a1, a2 = p.hash_a2;
    const int32_t L = (int32_t)p.L;

    int32_t*  s_c        = reinterpret_cast<int32_t*>(smem);
    uint32_t* s_q        = reinterpret_cast<uint32_t*>(s_c + S);
    uint32_t* s_win      = s_q + S;                                   // per-bucket winner tag of UpdateState
    int32_t*  s_miss_x   = reinterpret_cast<int32_t*>(s_win + S);
    uint16_t* s_miss_pos = reinterpret_cast<uint16_t*>(s_miss_x + Kp);
    uint16_t* s_dead     = s_miss_pos + Kp;
    uint16_t* s_bucket   = s_dead + Kp;                               // bit 15: a reusable bucket was found
    uint32_t* s_hist     = reinterpret_cast<uint32_t*>(s_bucket + Kp);
    uint32_t* s_scan_a   = s_hist + 128;
    uint32_t* s_scan_b   = s_scan_a + 40;
    const uint32_t priv_stride = nt + 4u;
    uint8_t*  s_priv     = L <= PRIV_HIST_MAX_L ? reinterpret_cast<uint8_t*>(s_scan_b + 40) : nullptr;

    const uint32_t ti = p.first + blockIdx.x, table = p.table_id[blockIdx.x];
    int32_t*  g_c = p.tok + (size_t)table * S;
    uint32_t* g_q = p.qword + (size_t)table * S;
    int8_t*   g_life = p.life + (size_t)table * S;
    const uint32_t spt = S >= nt ? S / nt : 1u, j0 = tid * spt;
    const bool own = j0 < S;
    const uint32_t ipt = (K + nt - 1) / nt, i0 = tid * ipt;

    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (p.t_range && threadIdx.x == 0) atomicMin(p.t_range, global_ns());
    const uint32_t epoch = p.flags ? __ldcg(p.epoch) : 0u;

    // ---- load the table; global pre-decay ----
    if (own)
        for (uint32_t k = 0; k < spt; ++k) {
            s_c[j0 + k] = __ldg(g_c + j0 + k);
            s_q[j0 + k] = __ldg(g_q + j0 + k);
            s_win[j0 + k] = 0;
        }
    if (s_priv)
        for (uint32_t i = tid; i < ((uint32_t)(L + 2) * priv_stride + 15u) / 16u; i += nt)
            reinterpret_cast<int4*>(s_priv)[i] = make_int4(0, 0, 0, 0);
    int32_t xs[MAX_IPT];
    load_ids(p.indices + (size_t)ti * p.n_q * K, i0, ipt, K, xs);
    __syncthreads();
    {
        uint32_t w0, w1;
        pack_life_bytes(s_q, j0, spt, own, w0, w1);
        unpack_life_bytes(s_q, j0, spt, own, decay4(w0, 1), decay4(w1, 1));
    }
    __syncthreads();

    uint32_t list_off = 0, sum_valid = 0, sum_miss = 0, sum_decay = 0;
    int2* list = p.miss_list + (size_t)ti * p.list_stride;

    for (uint32_t g = 0; g < p.n_q; ++g) {
        const size_t row = ((size_t)ti * p.n_q + g) * K;
        int32_t* O = p.slots + row;
        uint8_t* Hm = p.hit ? p.hit + row : nullptr;
        if (tid < 128) s_hist[tid] = 0;

        // ---- Probe (Eq. 8-11): at most R + 1 buckets; the full id is compared ----
        uint32_t missmask = 0, nmiss = 0, nvalid = 0;
        check_ids(xs, i0, ipt, K, p.id_limit[blockIdx.x], p.status);
#pragma unroll
        for (uint32_t k = 0; k < (uint32_t)MAX_IPT; ++k) {
            const uint32_t i = i0 + k;
            if (k < ipt && i < K) {
                const int32_t x = xs[k];
                if (x >= 0) {
                    ++nvalid;
                    uint32_t h = (a1 * (uint32_t)x) & (S - 1u);
                    const uint32_t d = ((a2 * (uint32_t)x) & (S - 1u)) | 1u;
                    int32_t j = -1;
                    for (uint32_t r = 0; r <= R; ++r) {
                        const uint32_t o = s_q[h] & (S - 1u);
                        if (s_c[o] == x) { j = (int32_t)o; break; }
                        if (r < R) h = (h + d) & (S - 1u);
                    }
                    if (j >= 0) {
                        reinterpret_cast<uint8_t*>(s_q)[4u * (uint32_t)j + 3u] = (uint8_t)L;    // lifetime <- L
                        O[i] = j;
                        if (Hm) Hm[i] = 1;
                    } else {
                        missmask |= 1u << k;
                        ++nmiss;
                    }
                } else {
                    O[i] = -1;
                    if (Hm) Hm[i] = 0;
                }
            }
        }
        uint32_t total;
        uint32_t off = block_excl_scan(nmiss | (nvalid << 16), s_scan_a, total) & 0xFFFFu;
        const uint32_t n_g = total & 0xFFFFu;
        sum_valid += total >> 16;
        sum_miss += n_g;
#pragma unroll
        for (uint32_t k = 0; k < (uint32_t)MAX_IPT; ++k) {
            if (missmask & (1u << k)) {
                s_miss_x[off] = xs[k];
                s_miss_pos[off] = (uint16_t)(i0 + k);
                ++off;
            }
        }
        if (g + 1 < p.n_q) load_ids(p.indices + row + K, i0, ipt, K, xs);
        if (tid == 0 && p.miss_count) p.miss_count[(size_t)ti * p.n_q + g] = (int32_t)n_g;
        if (n_g == 0) { __syncthreads(); publish_token(p, ti, table, g, 0, blockIdx.x, epoch); continue; }
        __syncthreads();

        // ---- CollectDead / decay until n_g slots are dead ----
        uint32_t w0, w1;
        pack_life_bytes(s_q, j0, spt, own, w0, w1);
        uint32_t sg0 = w0 & 0x80808080u, sg1 = w1 & 0x80808080u;
        uint32_t dtotal, d = 0;
        uint32_t doff = block_excl_scan(__popc(sg0) + __popc(sg1), s_scan_b, dtotal);
        if (dtotal < n_g) {
            count_lifetimes(w0, w1, spt, own, L, s_priv, priv_stride, s_hist);
            __syncthreads();
            uint32_t cum = 0;
            bool found = false;
            d = (uint32_t)L + 1u;
            for (uint32_t b = 0; b <= (uint32_t)L + 1u; ++b) {
                cum += s_hist[b];
                if (cum >= n_g) { d = b; found = true; break; }
            }
            if (!found && tid == 0) atomicOr(p.status, ST_NO_DEAD_SLOTS);
            w0 = decay4(w0, d);
            w1 = decay4(w1, d);
            unpack_life_bytes(s_q, j0, spt, own, w0, w1);
            sg0 = w0 & 0x80808080u; sg1 = w1 & 0x80808080u;
            doff = block_excl_scan(__popc(sg0) + __popc(sg1), s_scan_b, dtotal);
        }
#pragma unroll
        for (uint32_t k = 0; k < (uint32_t)MAX_SPT; ++k) {
            const uint32_t bit = k < 4 ? (sg0 >> (8 * k + 7)) & 1u : (sg1 >> (8 * (k - 4) + 7)) & 1u;
            if (bit) {
                if (doff < n_g) s_dead[doff] = (uint16_t)(j0 + k);
                ++doff;
            }
        }
        __syncthreads();
        const uint32_t n_take = n_g < dtotal ? n_g : dtotal;

        // ---- UpdateState (1): every miss looks for a reusable bucket on the table as it stands (Eq. 4) ----
        for (uint32_t k = tid; k < n_take; k += nt) {
            const int32_t x = s_miss_x[k];
            uint32_t h = (a1 * (uint32_t)x) & (S - 1u);
            const uint32_t dd = ((a2 * (uint32_t)x) & (S - 1u)) | 1u;
            uint32_t v = 0;
            for (uint32_t r = 0; r <= R; ++r) {
                const uint32_t qh = s_q[h], o = qh & (S - 1u);
                const uint32_t invalid = (qh >> 23) & 1u, fp = (qh >> m) & Fm;
                const int32_t life_o = (int32_t)(int8_t)(s_q[o] >> 24);
                v = invalid | (uint32_t)(life_o < 0) | (uint32_t)(fp != ((uint32_t)s_c[o] & Fm));
                if (v || r == R) break;
                h = (h + dd) & (S - 1u);
            }
            s_bucket[k] = (uint16_t)(h | (v ? 0x8000u : 0u));
        }
        __syncthreads();
        // ---- (2): ids and lifetimes go into the allocated slots ----
        for (uint32_t k = tid; k < n_take; k += nt) {
            const uint32_t j = s_dead[k], i = s_miss_pos[k];
            const int32_t x = s_miss_x[k];
            if (j < S && i < K) {
                s_c[j] = x;
                reinterpret_cast<uint8_t*>(s_q)[4u * j + 3u] = (uint8_t)L;
                O[i] = (int32_t)j;
                if (Hm) Hm[i] = 0;
                list[list_off + k] = make_int2(x, (int32_t)j);
                if (s_bucket[k] & 0x8000u) atomicMax(&s_win[s_bucket[k] & 0x7FFFu], ((g + 1u) << 16) | k);
            } else {
                list[list_off + k] = make_int2(-1, -1);
                atomicOr(p.status, ST_BAD_SLOT);
            }
        }
        __syncthreads();
        // ---- (3): the bucket word keeps its slot's lifetime, takes fingerprint and slot, becomes valid ----
        for (uint32_t k = tid; k < n_take; k += nt) {
            const uint32_t hb = s_bucket[k];
            if ((hb & 0x8000u) && s_win[hb & 0x7FFFu] == (((g + 1u) << 16) | k)) {
                const uint32_t h = hb & 0x7FFFu;
                s_q[h] = (s_q[h] & 0xFF000000u) | (((uint32_t)s_miss_x[k] & Fm) << m) | (uint32_t)s_dead[k];
            }
        }
        list_off += n_take;
        sum_decay += d;
        __syncthreads();
        publish_token(p, ti, table, g, n_take, blockIdx.x, epoch);
    }

    // ---- write back; speculative entries (id >= N) become empty ----
    const int32_t N = p.verified_len_dev ? __ldg(p.verified_len_dev + ti) : p.verified_len[blockIdx.x];
    if (own)
        for (uint32_t k = 0; k < spt; ++k) {
            const int32_t v = s_c[j0 + k];
            g_c[j0 + k] = v >= N ? -1 : v;
            g_q[j0 + k] = s_q[j0 + k];
            g_life[j0 + k] = (int8_t)(s_q[j0 + k] >> 24);
        }
    if (tid == 0) {
        SegDesc sd;
        sd.src_base = p.kv_base[blockIdx.x];
        sd.src_stride = p.kv_stride[blockIdx.x];
        sd.dst_base = reinterpret_cast<uint64_t>(p.buffer + (size_t)table * S * p.row_bytes);
        sd.count = list_off;
        sd.pad = 0;
        p.seg[ti] = sd;
        TableStats* st = p.stats + table;
        st->steps += 1;
        st->tokens += p.n_q;
        st->hits += sum_valid - sum_miss;
        st->misses += sum_miss;
        st->rows += list_off;
        st->extra_decays += sum_decay;
    }
    if (p.t_range) {
        __syncthreads();
        if (tid == 0) atomicMax(p.t_range + 1, global_ns());
    }
}

// "KV offload" comparator: every selected row moves, position (g, i) -> slot g*K + i.
__global__ void __launch_bounds__(256) avsg_all_k_prepare_kernel(const __grid_constant__ AllKParams p)
{
    __shared__ uint32_t s_valid;
    const uint32_t g = blockIdx.x, b = blockIdx.y, ti = p.first + b, K = p.K;
    const uint32_t table = p.table_id[b];
    if (threadIdx.x == 0) s_valid = 0;
    __syncthreads();
    const size_t row = ((size_t)ti * p.n_q + g) * K;
    int2* list = p.miss_list + (size_t)ti * p.list_stride + (size_t)g * K;
    uint32_t valid = 0;
    for (uint32_t i = threadIdx.x; i < K; i += blockDim.x) {
        int32_t x = __ldg(p.indices + row + i);
        if (x >= 0 && (uint32_t)x >= p.id_limit[b]) {             // beyond the table's host rows: not fetched
            atomicOr(p.status, ST_BAD_ID);
            x = -1;
        }
        const int32_t o = x >= 0 ? (int32_t)(g * K + i) : -1;
        p.slots[row + i] = o;
        if (p.hit) p.hit[row + i] = 0;
        list[i] = make_int2(x, o);
        valid += x >= 0;
    }
    valid = __reduce_add_sync(0xffffffffu, valid);
    if ((threadIdx.x & 31u) == 0 && valid) atomicAdd(&s_valid, valid);
    __syncthreads();
    if (threadIdx.x == 0) {
        if (p.miss_count) p.miss_count[(size_t)ti * p.n_q + g] = (int32_t)s_valid;
        TableStats* st = p.stats + table;
        atomicAdd(&st->tokens, 1ull);
        atomicAdd(&st->misses, (unsigned long long)s_valid);
        atomicAdd(&st->rows, (unsigned long long)s_valid);
        if (g == 0) {
            SegDesc sd;
            sd.src_base = p.kv_base[b];
            sd.src_stride = p.kv_stride[b];
            sd.dst_base = reinterpret_cast<uint64_t>(p.buffer + (size_t)table * p.S * p.row_bytes);
            sd.count = p.n_q * K;
            sd.pad = 0;
            p.seg[ti] = sd;
            atomicAdd(&st->steps, 1ull);
        }
    }
}

}  // namespace

size_t stage_one_smem_bytes(uint32_t S, uint32_t K, uint32_t L, bool direct)
{
    const size_t H = direct ? 0 : 2ull * S, Kp = (K + 7u) & ~7u;
    size_t n = S * 4 + H * 4 + Kp * 4 + H * 2 + Kp * 2 + Kp * 2 + S + (128 + 40 + 40 + 8) * 4;
    if ((int32_t)L <= PRIV_HIST_MAX_L) n += ((size_t)(L + 2) * (stage_one_threads(S, K) + 4) + 15) / 16 * 16;
    (void)direct;
    return n;
}

size_t stage_one_paper_smem_bytes(uint32_t S, uint32_t K, uint32_t L)
{
    const size_t Kp = (K + 7u) & ~7u;
    size_t n = S * 12 + Kp * 4 + Kp * 2 * 3 + (128 + 40 + 40) * 4;
    if ((int32_t)L <= PRIV_HIST_MAX_L) n += ((size_t)(L + 2) * (stage_one_threads(S, K) + 4) + 15) / 16 * 16;
    return n;
}

uint32_t stage_one_threads(uint32_t S, uint32_t K)
{
    (void)K;
    uint32_t t = S / 2;
    if (t < 128) t = 128;
    if (t > 1024) t = 1024;
    return t;
}

cudaError_t stage_one_prepare(size_t max_smem)
{
    const void* kernels[] = {
        reinterpret_cast<const void*>(avsg_stage_one_kernel<false, S1_MAX_TABLES, false>),
        reinterpret_cast<const void*>(avsg_stage_one_kernel<true, S1_MAX_TABLES, false>),
        reinterpret_cast<const void*>(avsg_stage_one_kernel<false, S1_BIG_TABLES, false>),
        reinterpret_cast<const void*>(avsg_stage_one_kernel<true, S1_BIG_TABLES, false>),
        reinterpret_cast<const void*>(avsg_stage_one_kernel<false, S1_MAX_TABLES, true>),
        reinterpret_cast<const void*>(avsg_stage_one_kernel<true, S1_MAX_TABLES, true>),
        reinterpret_cast<const void*>(avsg_stage_one_kernel<false, S1_BIG_TABLES, true>),
        reinterpret_cast<const void*>(avsg_stage_one_kernel<true, S1_BIG_TABLES, true>),
        reinterpret_cast<const void*>(avsg_stage_one_paper_kernel)};
    for (const void* k : kernels) {
        cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)max_smem);
        if (e != cudaSuccess) return e;
    }
    // The other kernels of this file are loaded now as well: the runtime loads a kernel at its first use, which may
    // have to wait for every stream of the device - forever, if a stream is waiting for something that very launch
    // would produce (a caller who arms a wait for a call's stage_one_done word before its first call).
    const void* others[] = {reinterpret_cast<const void*>(avsg_all_k_prepare_kernel),
                            reinterpret_cast<const void*>(avsg_reset_tables_kernel),
                            reinterpret_cast<const void*>(avsg_direct_index_from_state_kernel)};
    for (const void* k : others) {
        cudaFuncAttributes fa;
        cudaError_t e = cudaFuncGetAttributes(&fa, k);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

namespace {
template <int CAP>
cudaError_t launch_stage_one_t(const S1ParamsT<CAP>& p, uint32_t n_tables, cudaStream_t stream)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(n_tables);
    cfg.blockDim = dim3(stage_one_threads(p.S, p.K));
    const bool direct = p.where != nullptr;
    cfg.dynamicSmemBytes = stage_one_smem_bytes(p.S, p.K, p.L, direct);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (n_tables < p.n_launch)              // fewer blocks than tables: the blocks serve the tables in rounds
        return direct ? cudaLaunchKernelEx(&cfg, avsg_stage_one_kernel<true, CAP, true>, p)
                      : cudaLaunchKernelEx(&cfg, avsg_stage_one_kernel<false, CAP, true>, p);
    return direct ? cudaLaunchKernelEx(&cfg, avsg_stage_one_kernel<true, CAP, false>, p)
                  : cudaLaunchKernelEx(&cfg, avsg_stage_one_kernel<false, CAP, false>, p);
}
}  // namespace

cudaError_t launch_stage_one(const S1Params& p, uint32_t n_tables, cudaStream_t stream)
{
    if (p.qword == nullptr) return launch_stage_one_t(p, n_tables, stream);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(n_tables);
    cfg.blockDim = dim3(stage_one_threads(p.S, p.K));
    cfg.dynamicSmemBytes = stage_one_paper_smem_bytes(p.S, p.K, p.L);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, avsg_stage_one_paper_kernel, p);
}

cudaError_t launch_stage_one(const S1ParamsBig& p, uint32_t n_tables, cudaStream_t stream)
{
    return launch_stage_one_t(p, n_tables, stream);
}

cudaError_t launch_direct_index_from_state(const int32_t* tok, uint16_t* where, uint32_t first_table, uint32_t n_tables,
                                           uint32_t S, uint32_t max_context, cudaStream_t stream)
{
    const size_t n = (size_t)n_tables * S;
    const uint32_t blocks = (uint32_t)((n + 255) / 256 < 1184 ? (n + 255) / 256 : 1184);
    avsg_direct_index_from_state_kernel<<<blocks, 256, 0, stream>>>(tok, where, first_table, n_tables, S, max_context);
    return cudaGetLastError();
}

cudaError_t launch_reset_tables(const ResetParams& p, uint32_t n_tables, cudaStream_t stream)
{
    avsg_reset_tables_kernel<<<dim3(32, n_tables), 256, 0, stream>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_all_k_prepare(const AllKParams& p, uint32_t n_tables, cudaStream_t stream)
{
    avsg_all_k_prepare_kernel<<<dim3(p.n_q, n_tables), 256, 0, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace avsg
