// Stage Two of the AVSG operator: miss-only host -> device gather (Sec. 3.4).
//
// The step's miss list is segmented by table (token order, then position
// order inside a table).  Every thread block recomputes the exclusive prefix
// sum of the segment lengths, which gives N_miss, and takes a contiguous
// share of the work.  Work is counted in 16-byte units (row_bytes / 16 per
// row), so shares differ by at most one unit whatever the per-request miss
// counts are: the balanced partition of Eq. 6 at a finer grain than a row.
// Threads read the host rows in place (mapped pinned memory) with 16-byte
// loads and store them into the reserved slots.
//
// request_level = 1 gives the comparator S1 of App. D: block b serves
// segment b alone.
#include "avsg_kernels.cuh"

namespace avsg {
namespace {

constexpr int TILE_ROWS = 256;
constexpr int UNROLL = 4;

__device__ __forceinline__ uint32_t warp_incl_scan(uint32_t v, uint32_t lane)
{
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        uint32_t n = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= (uint32_t)o) v += n;
    }
    return v;
}

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

__global__ void __launch_bounds__(1024) avsg_transfer_kernel(const __grid_constant__ XferParams p)
{
    __shared__ uint32_t s_pref[XFER_MAX_SEG + 1];
    __shared__ uint32_t s_w[40];
    __shared__ uint64_t s_src[TILE_ROWS];
    __shared__ uint64_t s_dst[TILE_ROWS];

    const uint32_t tid = threadIdx.x, nt = blockDim.x;
    const uint32_t n_seg = p.n_seg;

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

    const uint32_t cpr = p.row_bytes >> 4;                    // 16-byte units per row
    uint64_t u0, u1;
    if (p.request_level) {
        u0 = (uint64_t)s_pref[blockIdx.x] * cpr;
        u1 = (uint64_t)s_pref[blockIdx.x + 1] * cpr;
    } else {
        const uint64_t U = (uint64_t)running * cpr, C = gridDim.x, c = blockIdx.x;
        const uint64_t q = U / C, r = U % C;
        u0 = c * q + (c < r ? c : r);
        u1 = u0 + q + (c < r ? 1u : 0u);
    }
    if (u0 >= u1) return;

    const uint64_t m_first = u0 / cpr, m_last = (u1 - 1) / cpr;     // rows this block touches
    for (uint64_t mt = m_first; mt <= m_last; mt += TILE_ROWS) {
        const uint32_t rows = (uint32_t)((m_last - mt + 1) < (uint64_t)TILE_ROWS ? (m_last - mt + 1) : TILE_ROWS);
        // resolve (host address, slot address) of the tile's rows
        for (uint32_t r = tid; r < rows; r += nt) {
            const uint32_t m = (uint32_t)(mt + r);
            uint32_t lo = 0, hi = n_seg;                           // largest lo with s_pref[lo] <= m
            while (hi - lo > 1) {
                const uint32_t mid = (lo + hi) >> 1;
                if (s_pref[mid] <= m) lo = mid; else hi = mid;
            }
            const uint32_t local = m - s_pref[lo];
            uint64_t src = 0, dst = 0;
            if (local < p.list_stride && m < running) {
                const int2 e = __ldg(p.miss_list + (size_t)lo * p.list_stride + local);
                const SegDesc sd = p.seg[lo];
                if (e.x >= 0 && e.y >= 0 && (uint32_t)e.y < p.S) {
                    src = sd.src_base + (uint64_t)(uint32_t)e.x * sd.src_stride;
                    dst = sd.dst_base + (uint64_t)(uint32_t)e.y * p.row_bytes;
                }
            } else {
                atomicOr(p.status, ST_BAD_SEGMENT);
            }
            s_src[r] = src;
            s_dst[r] = dst;
        }
        __syncthreads();
        const uint64_t tile0 = mt * cpr;
        const uint64_t t0 = u0 > tile0 ? u0 : tile0;
        const uint64_t tile1 = (mt + rows) * cpr;
        const uint64_t t1 = u1 < tile1 ? u1 : tile1;
        for (uint64_t ub = t0 + tid; ub < t1; ub += (uint64_t)nt * UNROLL) {
            int4 v[UNROLL];
            uint64_t dst[UNROLL];
#pragma unroll
            for (int k = 0; k < UNROLL; ++k) {
                const uint64_t u = ub + (uint64_t)k * nt;
                dst[k] = 0;
                if (u < t1) {
                    const uint32_t lu = (uint32_t)(u - tile0);
                    const uint32_t r = lu / cpr, c = lu - r * cpr;
                    const uint64_t src = s_src[r];
                    if (src) {
                        v[k] = *reinterpret_cast<const int4*>(src + 16ull * c);
                        dst[k] = s_dst[r] + 16ull * c;
                    }
                }
            }
#pragma unroll
            for (int k = 0; k < UNROLL; ++k)
                if (dst[k]) *reinterpret_cast<int4*>(dst[k]) = v[k];
        }
        __syncthreads();
    }
}

}  // namespace

cudaError_t launch_transfer(const XferParams& p, uint32_t blocks, uint32_t threads, cudaStream_t stream)
{
    avsg_transfer_kernel<<<blocks, threads, 0, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace avsg
