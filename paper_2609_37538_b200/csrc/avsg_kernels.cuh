// Internal declarations shared by the kernels and the C-ABI host code.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace avsg {

// Device status word: kernels OR one of these in when a bounded loop runs out
// or an index leaves its range; nothing ever traps.
enum : uint32_t {
    ST_PROBE_EXHAUSTED = 1u << 0,   // hash probe visited every bucket
    ST_NO_DEAD_SLOTS   = 1u << 1,   // fewer reclaimable slots than misses (Eq. 7 violated)
    ST_BAD_SLOT        = 1u << 2,   // slot / position index out of range
    ST_BAD_SEGMENT     = 1u << 3,   // transfer kernel could not resolve a miss
    ST_BAD_ID          = 1u << 4,   // an id beyond the table's host rows or the direct index (treated as padding)
    ST_WAIT_TIMEOUT    = 1u << 5,   // overlapped Stage Two: a bounded wait for Stage One ran out
};

// One segment of the step's miss list = the misses of one table, in token
// order then position order (Alg. 4 appends every token's misses to the step's transfer list).
struct SegDesc {
    uint64_t src_base;    // host KV base of the table (device-visible address)
    uint64_t src_stride;  // bytes between host rows
    uint64_t dst_base;    // device buffer base of the table
    uint32_t count;       // entries in the segment
    uint32_t pad;
};

// Wall-clock span of a grid for avsg_set_timing: every block reports its start and end (globaltimer, ns).
__device__ __forceinline__ unsigned long long global_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// Inclusive prefix sum over the lanes of a warp.
__device__ __forceinline__ uint32_t warp_incl_scan(uint32_t v, uint32_t lane)
{
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        uint32_t n = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= (uint32_t)o) v += n;
    }
    return v;
}

// Exclusive prefix sum over the block in thread order (the order-preserving compactions of Stage One, the miss
// prefix sums of Stage Two); s_w holds 33 words of shared memory.  Every thread of the block calls it.
__device__ __forceinline__ uint32_t block_excl_scan(uint32_t v, uint32_t* s_w, uint32_t& total)
{
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const uint32_t incl = warp_incl_scan(v, lane);
    if (lane == 31) s_w[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        uint32_t w = lane < nwarps ? s_w[lane] : 0u;
        uint32_t wi = warp_incl_scan(w, lane);
        s_w[lane] = wi - w;
        if (lane == 31) s_w[32] = wi;
    }
    __syncthreads();
    total = s_w[32];
    return incl - v + s_w[warp];
}

struct TableStats {
    unsigned long long steps, tokens, hits, misses, rows, extra_decays;
};

constexpr int S1_MAX_TABLES = 128;   // tables per Stage One launch with the small argument block (3.3 KB)
constexpr int S1_BIG_TABLES = 1024;  // ... with the large one (25 KB; kernel arguments may take up to 32 764 bytes)
constexpr int MAX_IPT = 8;           // ids per thread
constexpr int MAX_SPT = 8;           // slots per thread
constexpr int XFER_MAX_SEG = 2048;   // segments per Stage Two launch (prefix sums live in shared memory)

// The per-call host arrays travel as kernel arguments, CAP tables' worth of them: a call needs no staging copy.
template <int CAP>
struct S1ParamsT {
    int32_t*       tok;          // [num_tables][S]
    int8_t*        life;         // [num_tables][S]
    uint8_t*       buffer;       // [num_tables][S * row_bytes]
    TableStats*    stats;        // [num_tables]
    int2*          miss_list;    // [segments][list_stride]  (x, slot)
    SegDesc*       seg;          // [segments]
    uint32_t*      status;       // mapped host word
    const int32_t* indices;      // [n][n_q][K]
    int32_t*       slots;        // [n][n_q][K]
    uint8_t*       hit;          // [n][n_q][K] or null
    int32_t*       miss_count;   // [n][n_q] or null
    uint32_t S, logH, row_bytes, K, n_q, L;
    uint32_t first;              // index within the call of this launch's first table
    uint32_t n_launch;           // tables of this launch (the grid may have fewer blocks: a block then serves several)
    uint32_t round_size;         // overlapped Stage Two: tables per publication round (= grid size of Stage One)
    uint32_t list_stride;        // entries per segment of miss_list
    uint32_t max_context;        // direct index: entries per table
    uint16_t* where;             // direct index [num_tables][max_context], or null for the hash index
    uint32_t* qword;             // paper-literal mode: packed metadata words [num_tables][S], else null
    uint32_t probe_retries, hash_a1, hash_a2;   // paper-literal mode: R, a1, a2
    unsigned long long* t_range = nullptr;      // timing on: [0] earliest block start, [1] latest block end (ns)
    // overlapped Stage Two (null otherwise): flags[ti * n_q + g] = (epoch << 32) | misses of token g of the ti-th
    // table of the call, written when that token is placed; *epoch is the number of the current overlapped call
    // (the transfer grid advances it when it is through), so flags of earlier calls never look valid
    unsigned long long* flags = nullptr;
    const uint32_t*     epoch = nullptr;
    // calls with host buffers in that mode (null otherwise): the table that places the call's last token last
    // writes the call's sequence number to *done_seq, which the output download waits for
    unsigned long long* done_seq = nullptr;
    uint32_t*           done_ctr = nullptr;     // arrivals after the call's last token; wraps to zero at `expect`
    unsigned long long  host_seq = 0;
    uint32_t            expect = 0;             // tables of the call
    const int32_t* verified_len_dev = nullptr;  // [n] of the call: read instead of verified_len[] when set
    uint32_t table_id[CAP];
    int32_t  verified_len[CAP];
    uint32_t id_limit[CAP];      // ids >= this are not looked up or fetched (host rows of the table; direct index size)
    uint64_t kv_base[CAP];
    uint64_t kv_stride[CAP];
};
using S1Params = S1ParamsT<S1_MAX_TABLES>;
using S1ParamsBig = S1ParamsT<S1_BIG_TABLES>;
static_assert(sizeof(S1ParamsBig) <= 32764, "kernel argument block too large");

struct XferParams {
    const SegDesc* seg;
    const int2*    miss_list;
    uint32_t*      status;
    uint32_t n_seg, list_stride, row_bytes, request_level, S;
    // timing on: [0] earliest block start, [1] latest block end, [2] earliest start of a block's copy loop,
    // [3] earliest arrival of a block's first row, [4] earliest end of a block that copied something (ns)
    unsigned long long* t_range = nullptr;
};

constexpr int OVERLAP_MAX_TOKENS = 8;
constexpr uint32_t S1_ROUND_BLOCKS = 32;             // Stage One blocks of a call that is served in rounds
constexpr int OVERLAP_MAX_TABLES = S1_BIG_TABLES;   // one Stage One launch
constexpr uint32_t OVERLAP_SPIN_LIMIT = 1u << 18;   // polls before the wait gives up; a poll is an L2 round trip plus a 64 ns sleep, ~0.8 us measured: ~0.2 s

struct XferOverlapParams {       // Stage Two that starts on token g's misses while Stage One places token g+1
    const SegDesc* seg;          // bases written by Stage One before it publishes token 0
    const int2*    miss_list;
    uint32_t*      status;
    const unsigned long long* flags;   // [n][n_q] (epoch << 32) | miss count, written by Stage One per placed token
    uint32_t*      epoch;        // number of the current overlapped call; advanced by the last block of this grid
    uint32_t*      done;         // blocks of this grid that are through; wraps to zero by itself
    uint32_t n, n_q, list_stride, row_bytes, S;
    uint32_t round_size;         // tables per round (n: one round)
    uint32_t expect_extra;       // added to what a counter must reach: 0, or 1 for the wait-limit diagnostic
    unsigned long long* t_range = nullptr;
};

struct PosParams {               // comparator S2: equal top-K position partition
    const SegDesc* seg;          // per table: host base, stride, buffer base
    const int32_t* indices;      // [n][n_q*K]
    const int32_t* slots;        // [n][n_q*K] (written by Stage One)
    const uint8_t* hit;          // [n][n_q*K] (written by Stage One)
    uint32_t*      status;
    uint32_t n, per_table, row_bytes, S;     // per_table = n_q * K positions
};

struct AllKParams {
    const int32_t* indices;      // [n][n_q*K]
    int32_t*       slots;
    uint8_t*       hit;
    int32_t*       miss_count;
    int2*          miss_list;
    SegDesc*       seg;
    TableStats*    stats;
    uint8_t*       buffer;
    uint32_t*      status;
    uint32_t S, row_bytes, K, n_q, first, list_stride;
    uint32_t table_id[S1_MAX_TABLES];
    uint32_t id_limit[S1_MAX_TABLES];
    uint64_t kv_base[S1_MAX_TABLES];
    uint64_t kv_stride[S1_MAX_TABLES];
};

struct ResetParams {             // stream-ordered reset of some tables: empty, dead, counters and rows zeroed
    int32_t* tok; int8_t* life; uint8_t* buffer; TableStats* stats;
    uint32_t* qword;             // paper-literal mode, else null
    uint32_t S, row_bytes;
    uint32_t table_id[S1_MAX_TABLES];
};
cudaError_t launch_reset_tables(const ResetParams& p, uint32_t n_tables, cudaStream_t stream);

size_t stage_one_smem_bytes(uint32_t S, uint32_t K, uint32_t L, bool direct = false);
size_t stage_one_paper_smem_bytes(uint32_t S, uint32_t K, uint32_t L);
uint32_t stage_one_threads(uint32_t S, uint32_t K);
cudaError_t stage_one_prepare(size_t max_smem);
// n_blocks thread blocks serve the p.n_launch tables of the launch (one block per table unless the call runs in rounds)
cudaError_t launch_stage_one(const S1Params& p, uint32_t n_blocks, cudaStream_t stream);
cudaError_t launch_stage_one(const S1ParamsBig& p, uint32_t n_blocks, cudaStream_t stream);   // hash / direct index only
// Stage One with one table per thread-block cluster of C blocks (C = 2, 4 or 8; hash / direct index only)
uint32_t stage_one_cluster_threads(uint32_t S, uint32_t C);
size_t stage_one_cluster_smem_bytes(uint32_t S, uint32_t K, uint32_t L, uint32_t C, bool direct);
cudaError_t stage_one_cluster_prepare(size_t max_smem);
int stage_one_cluster_max_active(uint32_t S, uint32_t K, uint32_t L, uint32_t C, bool direct);   // after ..._prepare
cudaError_t launch_stage_one_cluster(const S1Params& p, uint32_t n_tables, uint32_t C, cudaStream_t stream);
cudaError_t launch_stage_one_cluster(const S1ParamsBig& p, uint32_t n_tables, uint32_t C, cudaStream_t stream);
cudaError_t launch_direct_index_from_state(const int32_t* tok, uint16_t* where, uint32_t first_table, uint32_t n_tables,
                                           uint32_t S, uint32_t max_context, cudaStream_t stream);
cudaError_t launch_all_k_prepare(const AllKParams& p, uint32_t n_tables, cudaStream_t stream);
cudaError_t launch_transfer(const XferParams& p, uint32_t blocks, uint32_t threads, cudaStream_t stream);
cudaError_t launch_transfer_overlap(const XferOverlapParams& p, uint32_t blocks, uint32_t threads, cudaStream_t stream);
cudaError_t launch_transfer_positions(const PosParams& p, uint32_t blocks, uint32_t threads, cudaStream_t stream);

// Optional output of a call (latency hiding, Sec. 6 with Sec. 3.6): which positions' rows come with THIS call's
// Stage Two.  A kernel of its own between Stage One and Stage Two, so that the Stage One kernels carry no code for
// an output few calls ask for (inside them it cost every call 1.7 us).  It also makes the call's "Stage One is
// done" announcement when the caller asked for both.
struct ArrivingParams {
    const SegDesc* seg;              // per table of the call: count = entries of its miss list
    const int2*    miss_list;        // [n][list_stride] (id, slot)
    const int32_t* slots;            // [n][per_table]
    uint8_t*       arriving;         // [n][per_table] out
    unsigned long long* done_seq;    // or null
    uint32_t*      done_ctr;         // wraps to zero at the grid size
    unsigned long long value;
    uint32_t n, per_table, S, list_stride;
    // overlapped Stage Two: Stage One's hand-over flags and the call number (see S1ParamsT), else null
    const unsigned long long* flags;
    const uint32_t* epoch;
    uint32_t n_q;
    uint32_t* status;
};
cudaError_t launch_arriving(const ArrivingParams& p, uint32_t blocks, cudaStream_t stream);
cudaError_t arriving_prepare();
cudaError_t transfer_prepare();

}  // namespace avsg
