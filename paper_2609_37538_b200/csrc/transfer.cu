// Stage Two of the AVSG operator: miss-only host -> device gather (Sec. 3.4).
//
// The step's miss list is segmented by table (token order, then position
// order inside a table).  Every thread block recomputes the exclusive prefix
// sum of the segment lengths, which gives N_miss, and takes floor(N_miss/C)
// or ceil(N_miss/C) consecutive misses (Eq. 6, C = number of blocks); inside
// a block the warps take rows round-robin.  One warp moves one row: its lanes
// read the host row in place (mapped pinned memory) with 16-byte loads, so a
// warp-wide load covers 512 contiguous bytes of ONE row, and store it into
// the reserved slot.  Keeping a warp inside one row matters: the host link
// is bound by the number of read requests, and 16-byte units that straddle
// two rows produce more, smaller requests (measured 43.5 vs 47.5 GB/s).
//
// request_level = 1 gives the comparator S1 of App. D: block b serves
// segment b alone.
//
// avsg_transfer_overlap_kernel is the same gather started per token while
// Stage One still runs (App. G, latency hiding; described at the kernel), and
// avsg_transfer_positions_kernel is the comparator S2 of App. D.
#include "avsg_kernels.cuh"

namespace avsg {
namespace {

constexpr int CHUNKS_PER_PASS = 4;     // 16-byte loads a lane keeps in flight (covers rows up to 2 KiB per pass)

// 16-byte global load / store in the order written (volatile asm statements keep their relative order).
__device__ __forceinline__ int4 ld16(uint64_t addr)
{
    int4 v;
    asm volatile("ld.global.v4.s32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(addr));
    return v;
}
__device__ __forceinline__ void st16(uint64_t addr, const int4& v)
{
    asm volatile("st.global.v4.s32 [%0], {%1, %2, %3, %4};" :: "l"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

// One warp moves one row: 16-byte loads from the (host) source, all issued before the 16-byte stores into the slot.
// Rows of up to 1 KiB (two loads per lane) take the short path, whose instruction order is fixed by hand: both
// loads of a lane are in flight together.
__device__ __forceinline__ void copy_row(uint64_t src, uint64_t dst, uint32_t cpr, uint32_t lane)
{
    if (cpr <= 64u) {
        const bool p0 = lane < cpr, p1 = lane + 32u < cpr;
        int4 a = make_int4(0, 0, 0, 0), b = make_int4(0, 0, 0, 0);
        if (p0) a = ld16(src + 16ull * lane);
        if (p1) b = ld16(src + 16ull * (lane + 32u));
        if (p0) st16(dst + 16ull * lane, a);
        if (p1) st16(dst + 16ull * (lane + 32u), b);
        return;
    }
    for (uint32_t c0 = lane; c0 < cpr; c0 += 32u * CHUNKS_PER_PASS) {
        int4 v[CHUNKS_PER_PASS];
#pragma unroll
        for (int k = 0; k < CHUNKS_PER_PASS; ++k) {
            const uint32_t c = c0 + 32u * k;
            if (c < cpr) v[k] = *reinterpret_cast<const int4*>(src + 16ull * c);
        }
#pragma unroll
        for (int k = 0; k < CHUNKS_PER_PASS; ++k) {
            const uint32_t c = c0 + 32u * k;
            if (c < cpr) *reinterpret_cast<int4*>(dst + 16ull * c) = v[k];
        }
    }
}

__global__ void __launch_bounds__(1024, 1) avsg_transfer_kernel(const __grid_constant__ XferParams p)
{
    __shared__ uint32_t s_pref[XFER_MAX_SEG + 1];
    __shared__ uint32_t s_w[40];

    const uint32_t tid = threadIdx.x, nt = blockDim.x, lane = tid & 31u;
    const uint32_t n_seg = p.n_seg;

    // Programmatic dependent launch: the blocks may already be resident while Stage One still runs; the miss
    // list is read only after that grid has completed.  The kernel after this one may start its prologue.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (p.t_range && tid == 0) atomicMin(p.t_range, global_ns());

    // global miss prefix sum (every block computes the same one)
    uint32_t running = 0;
    for (uint32_t base = 0; base < n_seg; base += nt) {
        const uint32_t i = base + tid;
        const uint32_t c = i < n_seg ? p.seg[i].count : 0u;
        uint32_t total;
        const uint32_t excl = block_excl_scan(c, s_w, total);
        if (i < n_seg) s_pref[i] = running + excl;
        running += total;
        __syncthreads();
    }
    if (tid == 0) s_pref[n_seg] = running;
    __syncthreads();

    uint32_t m0, m1;                                           // this block's share of the miss list
    if (p.request_level) {
        m0 = s_pref[blockIdx.x];
        m1 = s_pref[blockIdx.x + 1];
    } else {
        const uint32_t C = gridDim.x, c = blockIdx.x, q = running / C, r = running % C;
        m0 = c * q + (c < r ? c : r);
        m1 = m0 + q + (c < r ? 1u : 0u);
    }

    const uint32_t cpr = p.row_bytes >> 4;                     // 16-byte chunks per row
    bool first_row = p.t_range != nullptr;                     // timing: when the copy starts, when its first row is in
    if (first_row && tid == 0 && m1 > m0) atomicMin(p.t_range + 2, global_ns());
    for (uint32_t m = m0 + (tid >> 5); m < m1; m += nt >> 5) {
        uint32_t lo = 0, hi = n_seg;                           // largest lo with s_pref[lo] <= m
        while (hi - lo > 1) {
            const uint32_t mid = (lo + hi) >> 1;
            if (s_pref[mid] <= m) lo = mid; else hi = mid;
        }
        const uint32_t local = m - s_pref[lo];
        if (local >= p.list_stride) {
            if (lane == 0) atomicOr(p.status, ST_BAD_SEGMENT);
            continue;
        }
        const int2 e = __ldg(p.miss_list + (size_t)lo * p.list_stride + local);
        if (e.x < 0) continue;                                 // padding entry of the transfer-all-K comparator
        if (e.y < 0 || (uint32_t)e.y >= p.S) {
            if (lane == 0) atomicOr(p.status, ST_BAD_SLOT);
            continue;
        }
        const uint64_t src = __ldg(&p.seg[lo].src_base) + (uint64_t)(uint32_t)e.x * __ldg(&p.seg[lo].src_stride);
        const uint64_t dst = __ldg(&p.seg[lo].dst_base) + (uint64_t)(uint32_t)e.y * p.row_bytes;
        copy_row(src, dst, cpr, lane);
        if (first_row) {
            if (tid == 0) atomicMin(p.t_range + 3, global_ns());
            first_row = false;
        }
    }
    if (p.t_range) {
        __syncthreads();
        if (tid == 0) {
            const unsigned long long t = global_ns();
            atomicMax(p.t_range + 1, t);
            if (m1 > m0) atomicMin(p.t_range + 4, t);          // the earliest block to finish: the tail starts here
        }
    }
}

// Stage Two that overlaps Stage One (the latency-hiding direction of App. G).  The grid is launched with
// programmatic stream serialization and does NOT wait for Stage One to complete: its blocks become resident
// once every Stage One block has started, then wait - with a bound - until all tables of a round have
// placed token g (Stage One writes a flag per table and token, carrying the number of the call and the
// token's miss count, after making that token's miss-list entries visible; every thread polls one table's
// flag), cut that token's misses evenly over the blocks (Eq. 6 per round and token) and copy them while
// Stage One places the next token or the next round of tables.  A call is one round unless it has so many
// tables that Stage One, with a block per table, would take most of the SMs: then Stage One runs with
// round_size blocks that serve the tables round by round, and this grid follows them.  Every Stage One block
// is resident before this grid starts and never waits for it, so it always makes progress; if a wait still
// runs out the block sets ST_WAIT_TIMEOUT and stops copying.  Before leaving, every block waits for the
// completion of the Stage One grid, so that the completion of this grid implies it; the last block to leave
// then advances the call number, so that no flag of this call can be taken for one of the next - nothing has
// to be zeroed between calls, and the kernel arguments hold nothing that changes from call to call (a
// captured call can be replayed).  All reads of data written by the running Stage One go to L2 (ld.cg /
// acquire).
__global__ void __launch_bounds__(1024, 1) avsg_transfer_overlap_kernel(const __grid_constant__ XferOverlapParams p)
{
    __shared__ uint32_t s_pref[OVERLAP_MAX_TABLES + 1];
    __shared__ uint32_t s_off[OVERLAP_MAX_TABLES];
    __shared__ uint64_t s_src[OVERLAP_MAX_TABLES], s_stride[OVERLAP_MAX_TABLES], s_dst[OVERLAP_MAX_TABLES];
    __shared__ uint32_t s_w[40];

    const uint32_t tid = threadIdx.x, nt = blockDim.x, lane = tid & 31u;
    const uint32_t n = p.n, rounds = (n + p.round_size - 1u) / p.round_size;

    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (p.t_range && tid == 0) atomicMin(p.t_range, global_ns());
    // the number of this call: the previous overlapped call's grid advanced it before this call's Stage One,
    // which this grid was launched behind, could start
    uint32_t epoch;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(epoch) : "l"(p.epoch) : "memory");
    for (uint32_t i = tid; i < n; i += nt) s_off[i] = 0;
    __syncthreads();

    const uint32_t cpr = p.row_bytes >> 4;
    bool first_row = p.t_range != nullptr, copied = false, gave_up = false;
    for (uint32_t r = 0; r < rounds && !gave_up; ++r) {
        const uint32_t base = r * p.round_size;                        // tables [base, base + nr) of the call
        const uint32_t nr = n - base < p.round_size ? n - base : p.round_size;
        for (uint32_t g = 0; g < p.n_q; ++g) {
            // every thread waits for the flag of one table of the round (of several, if the block is small)
            int ok = 1;
            for (uint32_t i = tid; i < nr; i += nt) {
                const unsigned long long* f = p.flags + (size_t)(base + i) * p.n_q + g;
                unsigned long long v = 0;
                uint32_t spin = 0;
                for (; spin < OVERLAP_SPIN_LIMIT; ++spin) {
                    asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(f) : "memory");
                    if ((uint32_t)(v >> 32) == epoch + p.expect_extra) break;
                    __nanosleep(64);
                }
                if (spin == OVERLAP_SPIN_LIMIT) { ok = 0; atomicOr(p.status, ST_WAIT_TIMEOUT); break; }
                s_pref[i] = (uint32_t)v;                               // the table's miss count of this token
            }
            if (!__syncthreads_and(ok)) { gave_up = true; break; }     // same decision in every thread
            if (g == 0)                                                // a table's bases are published with its token 0
                for (uint32_t i = base + tid; i < base + nr; i += nt) {
                    s_src[i] = __ldcg(&p.seg[i].src_base);
                    s_stride[i] = __ldcg(&p.seg[i].src_stride);
                    s_dst[i] = __ldcg(&p.seg[i].dst_base);
                }

            // prefix sum of token g's miss counts over the tables of the round (the counts came with the flags)
            uint32_t running = 0;
            for (uint32_t b0 = 0; b0 < nr; b0 += nt) {
                const uint32_t i = b0 + tid;
                const uint32_t c = i < nr ? s_pref[i] : 0u;
                uint32_t total;
                const uint32_t excl = block_excl_scan(c, s_w, total);
                if (i < nr) s_pref[i] = running + excl;
                running += total;
                __syncthreads();
            }
            if (tid == 0) s_pref[nr] = running;
            __syncthreads();

            const uint32_t C = gridDim.x, cb = blockIdx.x, q = running / C, rem = running % C;
            const uint32_t m0 = cb * q + (cb < rem ? cb : rem);
            const uint32_t m1 = m0 + q + (cb < rem ? 1u : 0u);
            if (first_row && tid == 0 && m1 > m0) atomicMin(p.t_range + 2, global_ns());
            copied = copied || m1 > m0;
            for (uint32_t m = m0 + (tid >> 5); m < m1; m += nt >> 5) {
                uint32_t lo = 0, hi = nr;                              // largest lo with s_pref[lo] <= m
                while (hi - lo > 1) {
                    const uint32_t mid = (lo + hi) >> 1;
                    if (s_pref[mid] <= m) lo = mid; else hi = mid;
                }
                const uint32_t t = base + lo;                          // the table, within the call
                const uint32_t local = s_off[t] + (m - s_pref[lo]);    // entry of the table's miss list
                if (local >= p.list_stride) {
                    if (lane == 0) atomicOr(p.status, ST_BAD_SEGMENT);
                    continue;
                }
                const int2 e = __ldcg(p.miss_list + (size_t)t * p.list_stride + local);
                if (e.x < 0) continue;
                if (e.y < 0 || (uint32_t)e.y >= p.S) {
                    if (lane == 0) atomicOr(p.status, ST_BAD_SLOT);
                    continue;
                }
                const uint64_t src = s_src[t] + (uint64_t)(uint32_t)e.x * s_stride[t];
                const uint64_t dst = s_dst[t] + (uint64_t)(uint32_t)e.y * p.row_bytes;
                copy_row(src, dst, cpr, lane);
                if (first_row) {
                    if (tid == 0) atomicMin(p.t_range + 3, global_ns());
                    first_row = false;
                }
            }
            __syncthreads();
            for (uint32_t i = tid; i < nr; i += nt) s_off[base + i] += s_pref[i + 1] - s_pref[i];
            __syncthreads();
        }
    }
    unsigned long long t_copied = 0;
    if (p.t_range) {
        __syncthreads();
        t_copied = global_ns();
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (p.t_range && tid == 0) {
        atomicMax(p.t_range + 1, global_ns());                     // the block's end, the wait for Stage One included
        if (copied) atomicMin(p.t_range + 4, t_copied);
    }
    // Stage One is complete (the wait above), so no flag of this call will be written any more: the last block to
    // arrive here advances the call number (0 is never used: the flags start out as zero)
    __syncthreads();
    if (tid == 0 && atomicInc(p.done, gridDim.x - 1u) == gridDim.x - 1u) {
        const uint32_t next = epoch + 1u ? epoch + 1u : 1u;
        asm volatile("st.release.gpu.global.u32 [%0], %1;" :: "l"(p.epoch), "r"(next) : "memory");
    }
}

// Comparator S2 (App. D, Eq. 14): the n * N_q * K selected positions of the call are flattened and cut into
// gridDim.x near-equal contiguous ranges regardless of hit or miss; a block walks its range, one warp per
// position, and copies the row of every position that missed.  Work per block = misses in its range (Eq. 15).
__global__ void __launch_bounds__(1024) avsg_transfer_positions_kernel(const __grid_constant__ PosParams p)
{
    const uint32_t lane = threadIdx.x & 31u, warps = blockDim.x >> 5;
    const uint64_t P = (uint64_t)p.n * p.per_table, C = gridDim.x, c = blockIdx.x;
    const uint64_t begin = c * P / C, end = (c + 1) * P / C;
    const uint32_t cpr = p.row_bytes >> 4;
    for (uint64_t q = begin + (threadIdx.x >> 5); q < end; q += warps) {
        const int32_t x = __ldg(p.indices + q);
        if (x < 0 || __ldg(p.hit + q)) continue;                 // padding or hit: nothing to move
        const int32_t o = __ldg(p.slots + q);
        if (o < 0) continue;                                     // an id Stage One refused (beyond the host rows)
        if ((uint32_t)o >= p.S) {
            if (lane == 0) atomicOr(p.status, ST_BAD_SLOT);
            continue;
        }
        const uint32_t ti = (uint32_t)(q / p.per_table);
        const uint64_t src = __ldg(&p.seg[ti].src_base) + (uint64_t)(uint32_t)x * __ldg(&p.seg[ti].src_stride);
        const uint64_t dst = __ldg(&p.seg[ti].dst_base) + (uint64_t)(uint32_t)o * p.row_bytes;
        copy_row(src, dst, cpr, lane);
    }
}

}  // namespace

cudaError_t launch_transfer_positions(const PosParams& p, uint32_t blocks, uint32_t threads, cudaStream_t stream)
{
    avsg_transfer_positions_kernel<<<blocks, threads, 0, stream>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_transfer_overlap(const XferOverlapParams& p, uint32_t blocks, uint32_t threads, cudaStream_t stream)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(blocks);
    cfg.blockDim = dim3(threads);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, avsg_transfer_overlap_kernel, p);
}

cudaError_t launch_transfer(const XferParams& p, uint32_t blocks, uint32_t threads, cudaStream_t stream)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(blocks);
    cfg.blockDim = dim3(threads);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, avsg_transfer_kernel, p);
}

// Loads this file's kernels (see stage_one_prepare() on why that is not left to their first launch).
cudaError_t transfer_prepare()
{
    const void* kernels[] = {reinterpret_cast<const void*>(avsg_transfer_kernel),
                             reinterpret_cast<const void*>(avsg_transfer_overlap_kernel),
                             reinterpret_cast<const void*>(avsg_transfer_positions_kernel)};
    for (const void* k : kernels) {
        cudaFuncAttributes fa;
        cudaError_t e = cudaFuncGetAttributes(&fa, k);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

}  // namespace avsg
