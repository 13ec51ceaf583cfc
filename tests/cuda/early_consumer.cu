// A stand-in for an attention kernel that starts on the hits of a decode step before the missed rows have arrived
// (latency hiding, Sec. 6 of the paper).  Test code: it is compiled by tests/test_gpu_parity.py, not part of the
// library.
//
// It is launched on the SAME stream as avsg_step, right after it, with programmatic stream serialization.  The
// operator's kernels release their dependents as soon as their blocks run, so this kernel starts while Stage One
// and Stage Two are still at work - and only then: every block of both is resident by the time it begins, so its
// wait below is for kernels that are running, never for one that has yet to be scheduled.
//   phase 1  wait (bounded) for the word the call writes at the end of its Stage One (avsg_step_args.stage_one_done);
//            the slot table, the hit mask and the `arriving` mask are final: copy the first two out, and read the row
//            of the first position whose row is NOT arriving, i.e. was resident before the call (a hit alone does
//            not say that: a later token may hit a slot reserved earlier in this very call, Sec. 3.6)
//   phase 2  griddepcontrol.wait: everything before it on the stream, i.e. Stage Two, is complete and visible;
//            read the row of one MISSED position
// 32 blocks; every block waits for the word by itself, the first one also reads the rows and takes the time marks
// (GPU clock): its start, the word seen, phase 1 finished, Stage Two waited for.
#include <cuda_runtime.h>
#include <stdint.h>

namespace {

__device__ __forceinline__ unsigned long long now_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

__device__ __forceinline__ unsigned long long load_acquire(const unsigned long long* p)
{
    unsigned long long v;
    asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}

struct ConsumerArgs {
    const unsigned long long* word;
    unsigned long long value;
    const int32_t* ids;          // [n_pos] the call's ids, table 0 first
    const int32_t* slots;        // [n_pos] written by the call
    const uint8_t* hit;          // [n_pos] written by the call
    const uint8_t* arriving;     // [n_pos] written by the call: 1 = the row comes with this call's Stage Two
    uint32_t n_pos;              // positions of the whole call
    uint32_t n_pos_table0;       // positions of table 0 (rows are read from table 0's buffer only)
    const uint8_t* buffer0;      // table 0's rows
    uint32_t row_bytes;
    int32_t* slots_early;        // [n_pos] out
    uint8_t* hit_early;          // [n_pos] out
    uint8_t* hit_row;            // [row_bytes] out: the row of the first resident position of table 0, read in phase 1
    uint8_t* miss_row;           // [row_bytes] out: the row of the first arriving position, read in phase 2
    int32_t* picked;             // [2] out: the ids whose rows were read (-1: none)
    unsigned long long* t_marks; // [4] out: start, word seen, phase 1 done, Stage Two waited for
    uint32_t* status;            // out: 1 = the wait ran out
};

__global__ void __launch_bounds__(256) early_consumer_kernel(ConsumerArgs a)
{
    __shared__ int s_hit_pos, s_miss_pos, s_ok;
    const uint32_t tid = threadIdx.x;
    const bool first = blockIdx.x == 0;
    if (tid == 0) {
        if (first) a.t_marks[0] = now_ns();
        uint32_t spins = 0;
        s_ok = 1;
        while (load_acquire(a.word) != a.value) {
            if (++spins > (1u << 22)) { s_ok = 0; *a.status = 1; break; }
            __nanosleep(64);
        }
        if (first) a.t_marks[1] = now_ns();
        s_hit_pos = s_miss_pos = 0x7FFFFFFF;
    }
    __syncthreads();
    if (s_ok) {
        for (uint32_t i = blockIdx.x * blockDim.x + tid; i < a.n_pos; i += gridDim.x * blockDim.x) {
            a.slots_early[i] = __ldcg(a.slots + i);
            a.hit_early[i] = __ldcg(a.hit + i);
        }
        if (first) {
            for (uint32_t i = tid; i < a.n_pos_table0; i += blockDim.x) {       // table 0: first resident position,
                if (__ldcg(a.slots + i) < 0) continue;                           // first position whose row is arriving
                atomicMin(__ldcg(a.arriving + i) ? &s_miss_pos : &s_hit_pos, (int)i);
            }
            __syncthreads();
            if (tid == 0) {
                a.picked[0] = s_hit_pos != 0x7FFFFFFF ? a.ids[s_hit_pos] : -1;
                a.picked[1] = s_miss_pos != 0x7FFFFFFF ? a.ids[s_miss_pos] : -1;
            }
            if (s_hit_pos != 0x7FFFFFFF) {          // that row was placed by an earlier call: readable now
                const uint8_t* src = a.buffer0 + (size_t)__ldcg(a.slots + s_hit_pos) * a.row_bytes;
                for (uint32_t b = tid; b < a.row_bytes; b += blockDim.x) a.hit_row[b] = __ldcg(src + b);
            }
        }
    }
    __syncthreads();
    if (first && tid == 0) a.t_marks[2] = now_ns();      // phase 1 is done: everything it read was ready
    asm volatile("griddepcontrol.wait;" ::: "memory");   // Stage Two has finished: the missed rows are in
    if (first && tid == 0) a.t_marks[3] = now_ns();
    if (first && s_ok && s_miss_pos != 0x7FFFFFFF) {
        const uint8_t* src = a.buffer0 + (size_t)__ldcg(a.slots + s_miss_pos) * a.row_bytes;
        for (uint32_t b = tid; b < a.row_bytes; b += blockDim.x) a.miss_row[b] = __ldcg(src + b);
    }
}

}  // namespace

extern "C" int launch_early_consumer(const void* word, unsigned long long value, const void* ids, const void* slots,
                                     const void* hit, const void* arriving, uint32_t n_pos, uint32_t n_pos_table0,
                                     const void* buffer0,
                                     uint32_t row_bytes, void* slots_early, void* hit_early, void* hit_row,
                                     void* miss_row, void* picked, void* t_marks, void* status, void* stream)
{
    ConsumerArgs a;
    a.word = static_cast<const unsigned long long*>(word); a.value = value;
    a.ids = static_cast<const int32_t*>(ids); a.slots = static_cast<const int32_t*>(slots);
    a.hit = static_cast<const uint8_t*>(hit); a.arriving = static_cast<const uint8_t*>(arriving); a.n_pos = n_pos; a.n_pos_table0 = n_pos_table0;
    a.buffer0 = static_cast<const uint8_t*>(buffer0); a.row_bytes = row_bytes;
    a.slots_early = static_cast<int32_t*>(slots_early); a.hit_early = static_cast<uint8_t*>(hit_early);
    a.hit_row = static_cast<uint8_t*>(hit_row); a.miss_row = static_cast<uint8_t*>(miss_row);
    a.picked = static_cast<int32_t*>(picked);
    a.t_marks = static_cast<unsigned long long*>(t_marks); a.status = static_cast<uint32_t*>(status);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(32); cfg.blockDim = dim3(256); cfg.stream = static_cast<cudaStream_t>(stream);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return (int)cudaLaunchKernelEx(&cfg, early_consumer_kernel, a);
}
