// Device helpers shared by the Stage One kernels (single-block and cluster): packed lifetime arithmetic, the
// lifetime histogram, id loads, and the per-token publication of the overlapped Stage Two.
#pragma once
#include "avsg_kernels.cuh"

namespace avsg {

constexpr int32_t EMPTY = -1;
constexpr int32_t PRIV_HIST_MAX_L = 30;   // private byte-counter histogram up to this L (32 rows)

__device__ __forceinline__ uint32_t hash_id(int32_t x, uint32_t logH)
{
    return ((uint32_t)x * 2654435769u) >> (32u - logH);
}

// The lifetimes of the slots a thread owns, packed one signed byte each into
// two words; unused lanes carry 0x7F (never counted, never dead).
__device__ __forceinline__ void life_load(const int8_t* base, uint32_t j0, uint32_t spt, bool own,
                                          uint32_t& w0, uint32_t& w1)
{
    w0 = w1 = 0x7F7F7F7Fu;
    if (!own) return;
    if (spt == 8) { const uint2 v = *reinterpret_cast<const uint2*>(base + j0); w0 = v.x; w1 = v.y; }
    else if (spt == 4) { w0 = *reinterpret_cast<const uint32_t*>(base + j0); }
    else if (spt == 2) { w0 = 0x7F7F0000u | *reinterpret_cast<const uint16_t*>(base + j0); }
    else { w0 = 0x7F7F7F00u | (uint8_t)base[j0]; }
}

__device__ __forceinline__ void life_store(int8_t* base, uint32_t j0, uint32_t spt, bool own, uint32_t w0, uint32_t w1)
{
    if (!own) return;
    if (spt == 8) { *reinterpret_cast<uint2*>(base + j0) = make_uint2(w0, w1); }
    else if (spt == 4) { *reinterpret_cast<uint32_t*>(base + j0) = w0; }
    else if (spt == 2) { *reinterpret_cast<uint16_t*>(base + j0) = (uint16_t)w0; }
    else { base[j0] = (int8_t)(w0 & 0xFFu); }
}

// life <- max(life - d, -1) on four packed signed bytes
__device__ __forceinline__ uint32_t decay4(uint32_t w, uint32_t d)
{
    return __vmaxs4(__vsubss4(w, d * 0x01010101u), 0xFFFFFFFFu);
}

// The ids a thread handles for one token: positions i0 .. i0+ipt-1.
__device__ __forceinline__ void load_ids(const int32_t* X, uint32_t i0, uint32_t ipt, uint32_t K, int32_t (&xs)[MAX_IPT])
{
    if ((ipt & 3u) == 0 && (K & 3u) == 0 && ((reinterpret_cast<uintptr_t>(X) & 15u) == 0)) {
#pragma unroll
        for (uint32_t q = 0; q < (uint32_t)MAX_IPT / 4; ++q) {
            if (4 * q < ipt && i0 + 4 * q < K) {
                const int4 v = __ldg(reinterpret_cast<const int4*>(X + i0) + q);
                xs[4 * q] = v.x; xs[4 * q + 1] = v.y; xs[4 * q + 2] = v.z; xs[4 * q + 3] = v.w;
            }
        }
    } else if (ipt == 2 && (K & 1u) == 0 && ((reinterpret_cast<uintptr_t>(X) & 7u) == 0)) {
        if (i0 < K) {
            const int2 v = __ldg(reinterpret_cast<const int2*>(X + i0));
            xs[0] = v.x; xs[1] = v.y;
        }
    } else {
#pragma unroll
        for (uint32_t k = 0; k < (uint32_t)MAX_IPT; ++k)
            if (k < ipt && i0 + k < K) xs[k] = __ldg(X + i0 + k);
    }
}

// Ids at or beyond the table's host row count (or, with the direct index, beyond its index) are never read from
// host memory: they are reported in the status word and then handled like padding.
__device__ __forceinline__ void check_ids(int32_t (&xs)[MAX_IPT], uint32_t i0, uint32_t ipt, uint32_t K, uint32_t limit,
                                          uint32_t* status)
{
#pragma unroll
    for (uint32_t k = 0; k < (uint32_t)MAX_IPT; ++k)
        if (k < ipt && i0 + k < K && xs[k] >= 0 && (uint32_t)xs[k] >= limit) {
            atomicOr(status, ST_BAD_ID);
            xs[k] = -1;
        }
}

// Lifetime histogram of the table: s_hist[v + 1] = number of slots with lifetime v, v = -1 .. L.
// s_hist must be zero on entry.  w0/w1 are the thread's packed lifetimes (life_load).
__device__ __forceinline__ void count_lifetimes(uint32_t w0, uint32_t w1, uint32_t spt, bool own, int32_t L,
                                                uint8_t* s_priv, uint32_t priv_stride, uint32_t* s_hist)
{
    const uint32_t tid = threadIdx.x, nt = blockDim.x, lane = tid & 31u;
    if (s_priv) {
        // private byte counters: row = lifetime value + 1, column = thread; no atomics
        if (own) {
#pragma unroll
            for (uint32_t k = 0; k < (uint32_t)MAX_SPT; ++k) {
                if (k < spt) {
                    const uint32_t byte = ((k < 4 ? w0 >> (8 * k) : w1 >> (8 * (k - 4))) + 1u) & 0xFFu;   // value + 1
                    s_priv[byte * priv_stride + tid] += 1;
                }
            }
        }
        __syncthreads();
        // one warp per row: sum nt byte counters with dp4a and clear them for the next use
        const uint32_t words = nt >> 2;
        for (uint32_t row = tid >> 5; row <= (uint32_t)L + 1u; row += nt >> 5) {
            uint32_t* r = reinterpret_cast<uint32_t*>(s_priv + row * priv_stride);
            uint32_t acc = 0;
            for (uint32_t i = lane; i < words; i += 32u) {
                acc = __dp4a(r[i], 0x01010101u, acc);
                r[i] = 0;
            }
            acc = __reduce_add_sync(0xffffffffu, acc);
            if (lane == 0) s_hist[row] = acc;
        }
    } else {
        for (int32_t v = -1; v <= L; ++v) {
            const uint32_t vv = (uint32_t)(v & 0xFF) * 0x01010101u;
            uint32_t c = (__popc(__vcmpeq4(w0, vv)) + __popc(__vcmpeq4(w1, vv))) >> 3;
            c = __reduce_add_sync(0xffffffffu, c);
            if (lane == 0 && c) atomicAdd(&s_hist[v + 1], c);
        }
    }
}

// Overlapped Stage Two only (p.flags set): tells the transfer kernel, which is already resident, that token g of
// this table is placed - `count` more entries of the table's miss list are final.  Called by every thread of the
// block: the block meets after its list writes; one thread then fences (the barrier makes the fence cover the whole
// block's earlier writes, as in a grid-wide barrier) and writes the table's flag of token g: the call's number
// (read once when the kernel starts) in the upper half, the count in the lower.
template <typename P>
__device__ __forceinline__ void publish_token(const P& p, uint32_t ti, uint32_t table, uint32_t g, uint32_t count,
                                              uint32_t bt,      // bt: the table's index within this launch
                                              uint32_t epoch)
{
    const bool announce = p.done_seq && g + 1 == p.n_q;
    if (!p.flags && !announce) return;
    const uint32_t tid = threadIdx.x;
    if (tid == 0 && p.flags) {
        if (g == 0) {
            SegDesc sd;
            sd.src_base = p.kv_base[bt];
            sd.src_stride = p.kv_stride[bt];
            sd.dst_base = reinterpret_cast<uint64_t>(p.buffer + (size_t)table * p.S * p.row_bytes);
            sd.count = 0;
            sd.pad = 0;
            p.seg[ti] = sd;
        }
    }
    __syncthreads();
    if (tid == 0) {
        __threadfence();
        if (p.flags)
            *reinterpret_cast<volatile unsigned long long*>(p.flags + (size_t)ti * p.n_q + g) =
                ((unsigned long long)epoch << 32) | count;
        // calls that asked for it (host buffers in the overlapped mode, or a caller's own signal word): the table
        // that arrives last after the call's last token announces that every table of the call has written its
        // slot table, hit mask and miss counts.  The arrivals are counted in a word of their own that wraps to
        // zero by itself (atomicInc), whatever state the transfer kernel leaves the per-token counters in.
        if (announce && atomicInc(p.done_ctr, p.expect - 1u) == p.expect - 1u) {
            __threadfence();
            *reinterpret_cast<volatile unsigned long long*>(p.done_seq) = p.host_seq;
        }
    }
}


}  // namespace avsg
