// Stage One of the AVSG operator across a thread-block cluster: one table per cluster of C blocks (C = 1, 2, 4, 8).
//
// Same results as the single-block kernel (Algorithm 1 with the lifetime operations of Algorithm 3, the tokens of an
// iteration in order as in Algorithm 4, the end-of-step invalidation), for tables that do not fit one SM's shared
// memory (S up to 32768 slots) and with a shorter critical path for the ones that do.
//
// Block r of the cluster owns the slots [r S/C, (r+1) S/C) - their cached ids and lifetimes live in its shared
// memory for the step - and looks up the positions [r Kc, (r+1) Kc), Kc = ceil(K/C), of every token.  What a block
// needs from another one goes through distributed shared memory with plain ld / st / atom.shared::cluster (no
// multicast, no TMA):
//   * Match: the slot an index entry points at may belong to another block: its cached id is read, and on a hit its
//     lifetime is set to L, in that block's shared memory.  With the hash index (2S buckets, block r holds buckets
//     [r 2S/C, (r+1) 2S/C)) the probes read remote buckets the same way.
//   * Order-preserving compaction of the misses and of the dead slots (Eq. 12): a block prefix sum, then every block
//     sends its total to all blocks and a cluster barrier turns the totals into cluster-wide offsets.  Position
//     order is block order, then thread order, so "the k-th miss in position order" and "the k-th dead slot in slot
//     order" are well defined across blocks.
//   * Closed-form decay (the while-loop of Algorithm 1): when the dead slots do not cover the misses, every block
//     sends its lifetime histogram to all blocks; all compute the same d.
//   * Install: the OWNER of the k-th dead slot fetches the k-th miss (id and position) from the block that
//     compacted it and writes the id, the lifetime L, the slot-table entry, the transfer-list entry and the index.
// Three cluster barriers per token (match -> dead-slot scan -> install -> next token), one or two more when a decay
// is needed.  Every decision that changes the control flow (n_g = 0, decay or not, index rebuild) is taken on
// exchanged, cluster-wide values, so all blocks of a cluster reach the same barriers.
#include "avsg_kernels.cuh"
#include "stage_one_common.cuh"

namespace avsg {
namespace {

constexpr uint32_t MAX_CL = 8;          // largest cluster (the portable limit)

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ uint32_t cluster_rank()
{
    uint32_t r; asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r)); return r;
}
__device__ __forceinline__ uint32_t cluster_size()
{
    uint32_t r; asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r)); return r;
}
// the address of the same shared-memory location in block `rank` of the cluster
__device__ __forceinline__ uint32_t map_rank(uint32_t saddr, uint32_t rank)
{
    uint32_t r; asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank)); return r;
}
__device__ __forceinline__ int32_t ldc_s32(uint32_t a)
{
    int32_t v; asm volatile("ld.shared::cluster.s32 %0, [%1];" : "=r"(v) : "r"(a) : "memory"); return v;
}
__device__ __forceinline__ uint32_t ldc_u16(uint32_t a)
{
    uint16_t v; asm volatile("ld.shared::cluster.u16 %0, [%1];" : "=h"(v) : "r"(a) : "memory"); return v;
}
__device__ __forceinline__ void stc_u32(uint32_t a, uint32_t v)
{
    asm volatile("st.shared::cluster.u32 [%0], %1;" :: "r"(a), "r"(v) : "memory");
}
__device__ __forceinline__ void stc_u16(uint32_t a, uint32_t v)
{
    asm volatile("st.shared::cluster.u16 [%0], %1;" :: "r"(a), "h"((uint16_t)v) : "memory");
}
__device__ __forceinline__ void stc_u8(uint32_t a, uint32_t v)
{
    asm volatile("st.shared::cluster.u8 [%0], %1;" :: "r"(a), "r"(v) : "memory");
}
__device__ __forceinline__ int32_t casc_s32(uint32_t a, int32_t cmp, int32_t val)
{
    int32_t old;
    asm volatile("atom.shared::cluster.cas.b32 %0, [%1], %2, %3;" : "=r"(old) : "r"(a), "r"(cmp), "r"(val) : "memory");
    return old;
}
// All threads of all blocks of the cluster; earlier (distributed) shared-memory and global writes of the cluster
// are visible to every thread of the cluster afterwards.
__device__ __forceinline__ void cluster_sync()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// Shared-memory layout of one block (the same in every block of the cluster, so that a location's address in
// another block follows from the local one).
struct Layout {
    uint32_t tok, key, miss_x, val, miss_pos, life, hist, xhist, xch, scan_a, scan_b, fill, priv, total;
};
__host__ __device__ inline Layout make_layout(uint32_t S, uint32_t K, uint32_t L, uint32_t C, bool direct, uint32_t nt)
{
    const uint32_t Sc = S / C, Hc = direct ? 0u : 2u * Sc, Kc = (K + C - 1) / C, Kcp = (Kc + 7u) & ~7u;
    Layout o;
    uint32_t a = 0;
    o.tok = a;      a += Sc * 4;
    o.key = a;      a += Hc * 4;
    o.miss_x = a;   a += Kcp * 4;
    o.val = a;      a += Hc * 2;
    o.miss_pos = a; a += Kcp * 2;
    o.life = a;     a += (Sc + 15u) & ~15u;
    o.hist = a;     a += 128 * 4;
    o.xhist = a;    a += MAX_CL * 128 * 4;          // lifetime histograms of all blocks
    o.xch = a;      a += 4 * 2 * MAX_CL * 4;        // totals of all blocks: [kind][token parity][block]
    o.scan_a = a;   a += 40 * 4;
    o.scan_b = a;   a += 40 * 4;
    o.fill = a;     a += 16;
    o.priv = a;
    if ((int32_t)L <= PRIV_HIST_MAX_L) a += ((L + 2u) * (nt + 4u) + 15u) & ~15u;
    o.total = a;
    return o;
}

enum : uint32_t { XCH_MISS = 0, XCH_DEAD = 1, XCH_DEAD2 = 2, XCH_FILL = 3 };

template <bool DIRECT, int CAP>
__global__ void __launch_bounds__(1024, 1) avsg_stage_one_cluster_kernel(const __grid_constant__ S1ParamsT<CAP> p)
{
    extern __shared__ __align__(16) unsigned char smem[];
    const uint32_t S = p.S, K = p.K, tid = threadIdx.x, nt = blockDim.x, lane = tid & 31u;
    const int32_t L = (int32_t)p.L;
    const uint32_t rank = cluster_rank(), C = cluster_size();
    const uint32_t Sc = S / C, logSc = 31u - (uint32_t)__clz((int)Sc);
    const uint32_t Hc = DIRECT ? 0u : 2u * Sc, logHc = logSc + 1u, H = 2u * S;
    const uint32_t Kc = (K + C - 1) / C;
    const uint32_t k_base = rank * Kc;                                       // first position this block looks up
    const uint32_t Kl = k_base < K ? (K - k_base < Kc ? K - k_base : Kc) : 0u;   // how many
    const uint32_t j_base = rank * Sc;                                       // first slot this block owns

    const Layout lay = make_layout(S, K, p.L, C, DIRECT, nt);
    int32_t*  s_tok      = reinterpret_cast<int32_t*>(smem + lay.tok);
    int32_t*  s_key      = reinterpret_cast<int32_t*>(smem + lay.key);
    int32_t*  s_miss_x   = reinterpret_cast<int32_t*>(smem + lay.miss_x);
    uint16_t* s_val      = reinterpret_cast<uint16_t*>(smem + lay.val);
    uint16_t* s_miss_pos = reinterpret_cast<uint16_t*>(smem + lay.miss_pos);
    int8_t*   s_life     = reinterpret_cast<int8_t*>(smem + lay.life);
    uint32_t* s_hist     = reinterpret_cast<uint32_t*>(smem + lay.hist);
    uint32_t* s_xhist    = reinterpret_cast<uint32_t*>(smem + lay.xhist);
    uint32_t* s_xch      = reinterpret_cast<uint32_t*>(smem + lay.xch);
    uint32_t* s_scan_a   = reinterpret_cast<uint32_t*>(smem + lay.scan_a);
    uint32_t* s_scan_b   = reinterpret_cast<uint32_t*>(smem + lay.scan_b);
    uint32_t* s_fill     = reinterpret_cast<uint32_t*>(smem + lay.fill);
    const uint32_t priv_stride = nt + 4u;
    uint8_t*  s_priv     = L <= PRIV_HIST_MAX_L ? smem + lay.priv : nullptr;
    const uint32_t a_tok = smem_u32(s_tok), a_key = smem_u32(s_key), a_val = smem_u32(s_val), a_life = smem_u32(s_life),
                   a_mx = smem_u32(s_miss_x), a_mp = smem_u32(s_miss_pos), a_xch = smem_u32(s_xch),
                   a_xhist = smem_u32(s_xhist);

    const uint32_t bt = blockIdx.x / C;                   // table of this cluster within the launch
    const uint32_t ti = p.first + bt;                     // ... within the call
    const uint32_t table = p.table_id[bt];
    int32_t* g_tok = p.tok + (size_t)table * S + j_base;
    int8_t*  g_life = p.life + (size_t)table * S + j_base;

    const uint32_t spt = Sc >= nt ? Sc / nt : 1u;         // slots per thread, power of two <= 8
    const uint32_t j0 = tid * spt;                        // local slot number
    const bool own = j0 < Sc;
    const uint32_t ipt = (Kc + nt - 1) / nt;              // ids per thread, <= 8
    const uint32_t i0 = tid * ipt;                        // local position
    uint16_t* where = DIRECT ? p.where + (size_t)table * p.max_context : nullptr;
    const uint32_t id_limit = p.id_limit[bt];

    // cached id / lifetime byte of slot j (any block's)
    auto tok_of = [&](uint32_t j) { return ldc_s32(map_rank(a_tok + 4u * (j & (Sc - 1u)), j >> logSc)); };
    auto refresh = [&](uint32_t j) { stc_u8(map_rank(a_life + (j & (Sc - 1u)), j >> logSc), (uint32_t)L); };
    // sends v to slot [kind][parity][rank] of every block's exchange array
    auto send_total = [&](uint32_t kind, uint32_t parity, uint32_t v) {
        if (tid < C) stc_u32(map_rank(a_xch + 4u * ((kind * 2u + parity) * MAX_CL + rank), tid), v);
    };
    auto totals = [&](uint32_t kind, uint32_t parity, uint32_t& before, uint32_t& all) {
        before = all = 0;
        for (uint32_t q = 0; q < C; ++q) {
            const uint32_t v = s_xch[(kind * 2u + parity) * MAX_CL + q];
            if (q < rank) before += v;
            all += v;
        }
    };

    // hash index over the whole cluster: bucket b lives in block b / Hc
    auto find = [&](int32_t x) -> int32_t {
        uint32_t b = hash_id(x, logHc + (31u - (uint32_t)__clz((int)C)));
        for (uint32_t it = 0; it < H; ++it) {
            const uint32_t q = b >> logHc, l = b & (Hc - 1u);
            const int32_t k = ldc_s32(map_rank(a_key + 4u * l, q));
            if (k == x) {
                const uint32_t j = ldc_u16(map_rank(a_val + 2u * l, q));
                return tok_of(j) == x ? (int32_t)j : -1;      // a stale key: the id was reclaimed this step
            }
            if (k == EMPTY) return -1;
            b = (b + 1u) & (H - 1u);
        }
        atomicOr(p.status, ST_PROBE_EXHAUSTED);
        return -1;
    };
    auto insert = [&](int32_t x, uint32_t slot) {
        uint32_t b = hash_id(x, logHc + (31u - (uint32_t)__clz((int)C)));
        for (uint32_t it = 0; it < H; ++it) {
            const uint32_t q = b >> logHc, l = b & (Hc - 1u);
            const int32_t old = casc_s32(map_rank(a_key + 4u * l, q), EMPTY, x);
            if (old == EMPTY || old == x) { stc_u16(map_rank(a_val + 2u * l, q), slot); return; }
            b = (b + 1u) & (H - 1u);
        }
        atomicOr(p.status, ST_PROBE_EXHAUSTED);
    };
    // (re)builds the index from the cached ids; returns the cluster-wide number of occupied buckets
    auto build = [&]() -> uint32_t {
        if constexpr (!DIRECT)
            for (uint32_t i = tid; i < Hc / 4; i += nt)
                reinterpret_cast<int4*>(s_key)[i] = make_int4(EMPTY, EMPTY, EMPTY, EMPTY);
        if (tid == 0) *s_fill = 0;
        cluster_sync();                                   // every block's buckets are empty, every block's ids in place
        uint32_t live = 0;
        if (own)
            for (uint32_t k = 0; k < spt; ++k) {
                const int32_t x = s_tok[j0 + k];
                if (x >= 0) { insert(x, j_base + j0 + k); ++live; }
            }
        live = __reduce_add_sync(0xffffffffu, live);
        if (lane == 0 && live) atomicAdd(s_fill, live);
        __syncthreads();
        send_total(XCH_FILL, 0, *s_fill);
        cluster_sync();
        uint32_t before, all;
        totals(XCH_FILL, 0, before, all);
        return all;
    };

    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (p.t_range && tid == 0) atomicMin(p.t_range, global_ns());
    const uint32_t epoch = p.flags ? __ldcg(p.epoch) : 0u;      // the number of this overlapped call

    // ---- issue every global load first: this block's part of the table state and of the first token's ids ----
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
    load_ids(p.indices + (size_t)ti * p.n_q * K + k_base, i0, ipt, Kl, xs);

    if (s_priv)
        for (uint32_t i = tid; i < ((uint32_t)(L + 2) * priv_stride + 15u) / 16u; i += nt)
            reinterpret_cast<int4*>(s_priv)[i] = make_int4(0, 0, 0, 0);
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
    uint32_t fill_bound = 0;                              // hash index: occupied buckets (upper bound), cluster-wide
    if constexpr (!DIRECT) fill_bound = build();          // (two cluster barriers inside)
    else cluster_sync();                                  // every block's ids and lifetimes are in place

    uint32_t list_off = 0, sum_valid = 0, sum_miss = 0, sum_decay = 0;
    int2* list = p.miss_list + (size_t)ti * p.list_stride;

    for (uint32_t g = 0; g < p.n_q; ++g) {
        const uint32_t par = g & 1u;
        const size_t row = ((size_t)ti * p.n_q + g) * K;
        int32_t* O = p.slots + row;
        uint8_t* Hm = p.hit ? p.hit + row : nullptr;
        if (tid < 128) s_hist[tid] = 0;

        // ---- Probe, refresh hits to L, emit hit slots (Pass 1 + Pass 2) ----
        uint32_t missmask = 0, nmiss = 0, nvalid = 0;
        uint32_t cand[MAX_IPT];
        check_ids(xs, i0, ipt, Kl, id_limit, p.status);
        if (DIRECT) {
#pragma unroll
            for (uint32_t k = 0; k < (uint32_t)MAX_IPT; ++k) {   // all loads are issued before any is used
                cand[k] = 0xFFFFFFFFu;
                if (k < ipt && i0 + k < Kl && xs[k] >= 0) cand[k] = __ldcg(where + xs[k]) & (S - 1u);
            }
        }
#pragma unroll
        for (uint32_t k = 0; k < (uint32_t)MAX_IPT; ++k) {
            const uint32_t i = k_base + i0 + k;           // position within the token
            if (k < ipt && i0 + k < Kl) {
                const int32_t x = xs[k];
                if (x >= 0) {
                    ++nvalid;
                    int32_t j;
                    if (DIRECT) j = tok_of(cand[k]) == x ? (int32_t)cand[k] : -1;
                    else j = find(x);
                    if (j >= 0) {
                        refresh((uint32_t)j);
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
        // order-preserving compaction of the misses: t = x[not m]; block order, then thread order
        uint32_t total;
        uint32_t off = block_excl_scan(nmiss | (nvalid << 16), s_scan_a, total) & 0xFFFFu;
#pragma unroll
        for (uint32_t k = 0; k < (uint32_t)MAX_IPT; ++k) {
            if (missmask & (1u << k)) {
                s_miss_x[off] = xs[k];
                s_miss_pos[off] = (uint16_t)(k_base + i0 + k);
                ++off;
            }
        }
        send_total(XCH_MISS, par, total);
        // the next token's ids travel while this token's misses are placed
        if (g + 1 < p.n_q) load_ids(p.indices + row + K + k_base, i0, ipt, Kl, xs);
        cluster_sync();                                   // (1) hits refreshed everywhere, miss totals exchanged
        uint32_t m_before_packed, m_all_packed;
        totals(XCH_MISS, par, m_before_packed, m_all_packed);
        const uint32_t n_g = m_all_packed & 0xFFFFu;
        sum_valid += m_all_packed >> 16;
        sum_miss += n_g;
        if (rank == 0 && tid == 0 && p.miss_count) p.miss_count[(size_t)ti * p.n_q + g] = (int32_t)n_g;
        if (n_g == 0) {                                   // the same decision in every block of the cluster
            if (rank == 0) publish_token(p, ti, table, g, 0, bt, epoch);
            continue;
        }

        // ---- Pass 3: CollectDead; if fewer than n_g slots are dead, decay until enough are ----
        uint32_t w0, w1;
        life_load(s_life, j0, spt, own, w0, w1);
        uint32_t sg0 = w0 & 0x80808080u, sg1 = w1 & 0x80808080u;       // sign bits = dead slots
        uint32_t dloc, d = 0;
        uint32_t doff = block_excl_scan(__popc(sg0) + __popc(sg1), s_scan_b, dloc);
        send_total(XCH_DEAD, par, dloc);
        cluster_sync();                                   // (2) dead-slot totals exchanged
        uint32_t d_before, dtotal;
        totals(XCH_DEAD, par, d_before, dtotal);
        if (dtotal < n_g) {                               // same decision everywhere
            // the while-loop of Alg. 1 in closed form: d = fewest unit decays after which n_g slots are dead, read
            // off the histogram of the lifetimes of the whole table (every block sends its own to all blocks)
            count_lifetimes(w0, w1, spt, own, L, s_priv, priv_stride, s_hist);
            __syncthreads();
            for (uint32_t i = tid; i < C * ((uint32_t)L + 2u); i += nt) {
                const uint32_t q = i / ((uint32_t)L + 2u), b = i % ((uint32_t)L + 2u);
                stc_u32(map_rank(a_xhist + 4u * (rank * 128u + b), q), s_hist[b]);
            }
            cluster_sync();
            uint32_t cum = 0;
            bool found = false;
            d = (uint32_t)L + 1u;
            for (uint32_t b = 0; b <= (uint32_t)L + 1u; ++b) {   // bin b counts lifetime b-1; dead after b decays
                for (uint32_t q = 0; q < C; ++q) cum += s_xhist[q * 128u + b];
                if (cum >= n_g) { d = b; found = true; break; }
            }
            if (!found && rank == 0 && tid == 0) atomicOr(p.status, ST_NO_DEAD_SLOTS);
            w0 = decay4(w0, d);
            w1 = decay4(w1, d);
            life_store(s_life, j0, spt, own, w0, w1);
            sg0 = w0 & 0x80808080u; sg1 = w1 & 0x80808080u;
            doff = block_excl_scan(__popc(sg0) + __popc(sg1), s_scan_b, dloc);
            send_total(XCH_DEAD2, par, dloc);
            cluster_sync();
            totals(XCH_DEAD2, par, d_before, dtotal);
        }

        // ---- install: the owner of the k-th dead slot (slot order) takes the k-th miss (position order) ----
        const bool rebuild = !DIRECT && fill_bound + n_g > (H / 4u) * 3u;
        const uint32_t n_take = n_g < dtotal ? n_g : dtotal;
        uint32_t kk = d_before + doff;                    // cluster-wide rank of this thread's first dead slot
#pragma unroll
        for (uint32_t k = 0; k < (uint32_t)MAX_SPT; ++k) {
            const uint32_t bit = k < 4 ? (sg0 >> (8 * k + 7)) & 1u : (sg1 >> (8 * (k - 4) + 7)) & 1u;
            if (bit) {
                if (kk < n_take) {
                    // the block that compacted miss kk, and the miss's place in its list
                    uint32_t q = 0, base = 0;
                    for (; q + 1 < C; ++q) {
                        const uint32_t c = s_xch[(XCH_MISS * 2u + par) * MAX_CL + q] & 0xFFFFu;
                        if (kk < base + c) break;
                        base += c;
                    }
                    const int32_t x = ldc_s32(map_rank(a_mx + 4u * (kk - base), q));
                    const uint32_t i = ldc_u16(map_rank(a_mp + 2u * (kk - base), q));
                    const uint32_t jl = j0 + k, j = j_base + jl;
                    if (i < K) {
                        s_tok[jl] = x;
                        s_life[jl] = (int8_t)L;
                        O[i] = (int32_t)j;
                        if (Hm) Hm[i] = 0;
                        list[list_off + kk] = make_int2(x, (int32_t)j);
                        if (DIRECT) __stcg(where + x, (uint16_t)j);
                        else if (!rebuild) insert(x, j);
                    } else {
                        list[list_off + kk] = make_int2(-1, -1);         // Stage Two skips it
                        atomicOr(p.status, ST_BAD_SLOT);
                    }
                }
                ++kk;
            }
        }
        list_off += n_take;
        sum_decay += d;
        if (!rebuild) {
            fill_bound += n_g;
            cluster_sync();                               // (3) the new ids are visible to every block's next lookups
        } else if constexpr (!DIRECT) {
            fill_bound = build();
        }
        if (rank == 0) publish_token(p, ti, table, g, n_take, bt, epoch);
    }

    // ---- write this block's slots back; speculative entries (id >= N) become empty (Alg. 4) ----
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
    if (rank == 0 && tid == 0) {
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
    if (p.t_range) {
        __syncthreads();
        if (tid == 0) atomicMax(p.t_range + 1, global_ns());
    }
    // no block leaves while another one may still read its shared memory
    cluster_sync();
}

}  // namespace

uint32_t stage_one_cluster_threads(uint32_t S, uint32_t C)
{
    uint32_t t = S / C / 4;
    if (t < 128) t = 128;
    if (t > 1024) t = 1024;
    return t;
}

size_t stage_one_cluster_smem_bytes(uint32_t S, uint32_t K, uint32_t L, uint32_t C, bool direct)
{
    return make_layout(S, K, L, C, direct, stage_one_cluster_threads(S, C)).total;
}

cudaError_t stage_one_cluster_prepare(size_t max_smem)
{
    const void* kernels[] = {
        reinterpret_cast<const void*>(avsg_stage_one_cluster_kernel<false, S1_MAX_TABLES>),
        reinterpret_cast<const void*>(avsg_stage_one_cluster_kernel<true, S1_MAX_TABLES>),
        reinterpret_cast<const void*>(avsg_stage_one_cluster_kernel<false, S1_BIG_TABLES>),
        reinterpret_cast<const void*>(avsg_stage_one_cluster_kernel<true, S1_BIG_TABLES>)};
    for (const void* k : kernels) {
        cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)max_smem);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

namespace {
template <int CAP>
cudaError_t launch_cluster_t(const S1ParamsT<CAP>& p, uint32_t n_tables, uint32_t C, cudaStream_t stream)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(n_tables * C);
    cfg.blockDim = dim3(stage_one_cluster_threads(p.S, C));
    const bool direct = p.where != nullptr;
    cfg.dynamicSmemBytes = stage_one_cluster_smem_bytes(p.S, p.K, p.L, C, direct);
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = C;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return direct ? cudaLaunchKernelEx(&cfg, avsg_stage_one_cluster_kernel<true, CAP>, p)
                  : cudaLaunchKernelEx(&cfg, avsg_stage_one_cluster_kernel<false, CAP>, p);
}
}  // namespace

// How many clusters of this shape the device can hold at once (0: the shape cannot be launched at all).
int stage_one_cluster_max_active(uint32_t S, uint32_t K, uint32_t L, uint32_t C, bool direct)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(C);
    cfg.blockDim = dim3(stage_one_cluster_threads(S, C));
    cfg.dynamicSmemBytes = stage_one_cluster_smem_bytes(S, K, L, C, direct);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = C;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int n = 0;
    const cudaError_t e = direct
        ? cudaOccupancyMaxActiveClusters(&n, avsg_stage_one_cluster_kernel<true, S1_MAX_TABLES>, &cfg)
        : cudaOccupancyMaxActiveClusters(&n, avsg_stage_one_cluster_kernel<false, S1_MAX_TABLES>, &cfg);
    if (e != cudaSuccess) { cudaGetLastError(); return 0; }
    return n;
}

cudaError_t launch_stage_one_cluster(const S1Params& p, uint32_t n_tables, uint32_t C, cudaStream_t stream)
{
    return launch_cluster_t(p, n_tables, C, stream);
}

cudaError_t launch_stage_one_cluster(const S1ParamsBig& p, uint32_t n_tables, uint32_t C, cudaStream_t stream)
{
    return launch_cluster_t(p, n_tables, C, stream);
}

}  // namespace avsg
