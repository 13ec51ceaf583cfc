// The optional `arriving` output of avsg_step (Sec. 3.6 read with Sec. 6): for every position of the call, whether
// its row comes with THIS call's Stage Two or was resident before the call.
//
// A consumer that wants to start on the resident rows while the missed ones still travel cannot take the hit mask
// for that: with several tokens per iteration a later token may hit a slot that an earlier token of the same call
// has just reserved, and that row is still on its way.  A row is on its way exactly when its slot is the destination
// of an entry of the table's miss list - the position's own entry if it missed, or the earlier token's.
//
// One kernel between Stage One and Stage Two.  It releases its dependents at once, so that an overlapped transfer
// grid launched behind it is resident while Stage One runs, as without it.  When does it know that a table is
// placed?  With Stage Two after Stage One: when the Stage One grid has completed (griddepcontrol.wait).  With the
// overlapped Stage Two it reads the hand-over flags Stage One publishes per table and token, like the transfer grid
// does: measured, a dependent grid sees Stage One's COMPLETION only 40-50 us late while the transfer grid's host
// reads are in flight, whereas a flag is seen within a microsecond.  Every block of Stage One is resident before
// this grid starts (it is launched behind it with programmatic serialization), and the wait is bounded.
#include "avsg_kernels.cuh"

namespace avsg {
namespace {

__global__ void __launch_bounds__(512) avsg_arriving_kernel(const __grid_constant__ ArrivingParams p)
{
    extern __shared__ uint32_t s_bits[];                 // one bit per slot of the table at hand
    __shared__ uint32_t s_count;
    __shared__ int s_ok;
    const uint32_t tid = threadIdx.x, nt = blockDim.x, words = (p.S + 31u) / 32u;

    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    uint32_t epoch = 0;
    if (p.flags) {
        // the number of this overlapped call: final before Stage One, which this grid was launched behind, started
        asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(epoch) : "l"(p.epoch) : "memory");
    } else {
        asm volatile("griddepcontrol.wait;" ::: "memory");   // Stage One is complete: slot tables and lists are final
    }
    const bool vec = (p.per_table & 3u) == 0 && (reinterpret_cast<uint64_t>(p.slots) & 15u) == 0 &&
                     (reinterpret_cast<uint64_t>(p.arriving) & 3u) == 0;

    for (uint32_t ti = blockIdx.x; ti < p.n; ti += gridDim.x) {
        for (uint32_t w = tid; w < words; w += nt) s_bits[w] = 0;
        if (tid == 0) {
            s_ok = 1;
            if (p.flags) {
                // the table's last token is placed: its slot table is final, and so are the list entries the flags count
                uint32_t count = 0;
                for (uint32_t g = p.n_q; g-- > 0 && s_ok;) {          // last token first: the others are there by then
                    const unsigned long long* f = p.flags + (size_t)ti * p.n_q + g;
                    unsigned long long v = 0;
                    uint32_t spin = 0;
                    for (; spin < OVERLAP_SPIN_LIMIT; ++spin) {
                        asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(f) : "memory");
                        if ((uint32_t)(v >> 32) == epoch) break;
                        __nanosleep(64);
                    }
                    if (spin == OVERLAP_SPIN_LIMIT) { s_ok = 0; atomicOr(p.status, ST_WAIT_TIMEOUT); }
                    count += (uint32_t)v;
                }
                s_count = count;
            } else {
                s_count = p.seg[ti].count;
            }
        }
        __syncthreads();
        if (s_ok) {
            const int2* list = p.miss_list + (size_t)ti * p.list_stride;
            const uint32_t count = s_count < p.list_stride ? s_count : p.list_stride;
            for (uint32_t k = tid; k < count; k += nt) {
                const int32_t j = __ldcg(&list[k]).y;
                if (j >= 0 && (uint32_t)j < p.S) atomicOr(&s_bits[(uint32_t)j >> 5], 1u << (j & 31));
            }
            __syncthreads();
            const int32_t* slots = p.slots + (size_t)ti * p.per_table;
            uint8_t* out = p.arriving + (size_t)ti * p.per_table;
            auto coming = [&](int32_t j) -> uint32_t {
                return (j >= 0 && (uint32_t)j < p.S && ((s_bits[(uint32_t)j >> 5] >> (j & 31)) & 1u)) ? 1u : 0u;
            };
            if (vec) {
                for (uint32_t i = tid; i < p.per_table / 4u; i += nt) {
                    const int4 j = __ldcg(reinterpret_cast<const int4*>(slots) + i);
                    reinterpret_cast<uint32_t*>(out)[i] = coming(j.x) | coming(j.y) << 8 | coming(j.z) << 16 | coming(j.w) << 24;
                }
            } else {
                for (uint32_t i = tid; i < p.per_table; i += nt) out[i] = (uint8_t)coming(__ldcg(slots + i));
            }
        }
        __syncthreads();                                 // the bits are cleared again for the block's next table
    }
    // the block that finishes last announces that the call's Stage One outputs, this one included, are final
    if (tid == 0 && p.done_seq) {
        __threadfence();
        if (atomicInc(p.done_ctr, gridDim.x - 1u) == gridDim.x - 1u) {
            __threadfence();
            *reinterpret_cast<volatile unsigned long long*>(p.done_seq) = p.value;
        }
    }
}

}  // namespace

cudaError_t launch_arriving(const ArrivingParams& p, uint32_t blocks, cudaStream_t stream)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(blocks < p.n ? blocks : p.n);
    cfg.blockDim = dim3(512);
    cfg.dynamicSmemBytes = ((p.S + 31u) / 32u) * 4u;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, avsg_arriving_kernel, p);
}

// Loads the kernel (see stage_one_prepare() on why that is not left to its first launch).
cudaError_t arriving_prepare()
{
    cudaFuncAttributes fa;
    return cudaFuncGetAttributes(&fa, reinterpret_cast<const void*>(avsg_arriving_kernel));
}

}  // namespace avsg
