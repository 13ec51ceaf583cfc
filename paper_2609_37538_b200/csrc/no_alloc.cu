// avsg_step_noalloc: the decode step for callers that cannot allocate.
//
// Serving engines commonly claim all free device memory for their own pool at
// start-up, so a later cudaMalloc fails; other callers sit on a latency-
// critical path where cudaMalloc (which may synchronise the whole device) is
// not acceptable.  Such callers keep the table state (ids, lifetimes, KV
// rows) in memory they own and pass it in; what the step needs beyond its
// inputs and outputs - the miss list handed from Stage One to Stage Two, the
// per-table segment descriptors, counters and the status word - lives in the
// fixed device array below, which every GPU that loads this library holds
// until the process exits.
//
// This file calls no cudaMalloc / cudaFree / cudaHostAlloc and no library
// routine that allocates.
#include <mutex>
#include <stddef.h>
#include <string.h>

#include "avsg.h"
#include "avsg_kernels.cuh"

using namespace avsg;

namespace {

struct NoAllocScratch {
    uint32_t   status[64];                                   // word 0: device status
    SegDesc    seg[AVSG_NOALLOC_MAX_TABLES];
    TableStats stats[AVSG_NOALLOC_MAX_TABLES];
    int2       list[AVSG_NOALLOC_MAX_IDS];                   // (host position, slot) per miss
};

// About 1 MiB per GPU.  In host code this name is only a stand-in for the
// symbol, not a device address: the address is asked for once per device.
static __device__ __align__(256) unsigned char g_noalloc_scratch[sizeof(NoAllocScratch)];

constexpr int MAX_DEVICES = 64;
std::mutex g_setup_mutex;
NoAllocScratch* g_scratch_addr[MAX_DEVICES] = {nullptr};
int g_sm_count[MAX_DEVICES] = {0};
int g_max_smem[MAX_DEVICES] = {0};

// Once per device, with that device current: device address of the scratch
// array, device limits, and the Stage One kernel's shared-memory limit.
int setup_device(int dev, NoAllocScratch** out)
{
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_addr[dev]) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess || !ptr) { cudaGetLastError(); return AVSG_ECUDA; }
        if (cudaDeviceGetAttribute(&g_sm_count[dev], cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&g_max_smem[dev], cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess ||
            stage_one_prepare((size_t)g_max_smem[dev]) != cudaSuccess || transfer_prepare() != cudaSuccess) {
            cudaGetLastError();
            return AVSG_ECUDA;
        }
        g_scratch_addr[dev] = static_cast<NoAllocScratch*>(ptr);
    }
    *out = g_scratch_addr[dev];
    return AVSG_OK;
}

bool pow2(uint32_t v) { return v && !(v & (v - 1)); }

}  // namespace

extern "C" int avsg_step_noalloc(const avsg_noalloc_args* a, void* cuda_stream)
{
    if (!a) return AVSG_EINVAL;
    if (a->n == 0 || a->n_tokens == 0 || a->topk == 0) return AVSG_EINVAL;
    if (!pow2(a->buffer_slots) || a->buffer_slots < 32 || a->row_bytes == 0 || a->row_bytes % 16) return AVSG_EINVAL;
    if (a->max_lifetime < 1 || a->max_lifetime > 126) return AVSG_EINVAL;
    if (!a->tok || !a->life || !a->buffer || !a->indices || !a->kv_base || !a->verified_len || !a->slots) return AVSG_EINVAL;
    // the fixed scratch bounds what one call may carry
    if (a->n > AVSG_NOALLOC_MAX_TABLES || a->buffer_slots > 8192) return AVSG_EUNSUPPORTED;
    if ((uint64_t)a->n * a->n_tokens * a->topk > AVSG_NOALLOC_MAX_IDS) return AVSG_EUNSUPPORTED;
    if ((uint64_t)a->n_tokens * a->topk > a->buffer_slots) return AVSG_ECAPACITY;          // Eq. 7

    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return AVSG_ECUDA;
    NoAllocScratch* sc = nullptr;
    int rc = setup_device(dev, &sc);
    if (rc != AVSG_OK) return rc;
    if (stage_one_smem_bytes(a->buffer_slots, a->topk, (uint32_t)a->max_lifetime) > (size_t)g_max_smem[dev])
        return AVSG_EUNSUPPORTED;

    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const uint32_t list_stride = a->n_tokens * a->topk;

    S1Params p;
    p.tok = a->tok; p.life = a->life; p.buffer = static_cast<uint8_t*>(a->buffer);
    p.stats = sc->stats; p.miss_list = sc->list; p.seg = sc->seg; p.status = sc->status;
    p.indices = a->indices; p.slots = a->slots; p.hit = a->hit; p.miss_count = a->miss_count;
    p.S = a->buffer_slots; p.row_bytes = a->row_bytes; p.K = a->topk; p.n_q = a->n_tokens;
    p.L = (uint32_t)a->max_lifetime; p.first = 0; p.list_stride = list_stride;
    p.n_launch = a->n; p.round_size = a->n;
    p.where = nullptr; p.max_context = 0;
    p.qword = nullptr; p.probe_retries = 0; p.hash_a1 = 0; p.hash_a2 = 0;
    p.logH = 1;
    while ((1u << p.logH) < 2u * a->buffer_slots) ++p.logH;
    for (uint32_t i = 0; i < a->n; ++i) {
        const void* base = a->kv_base[i];
        if (!base || (reinterpret_cast<uint64_t>(base) & 15u)) return AVSG_EINVAL;
        if (a->row_stride && (a->row_stride[i] % 16 || a->row_stride[i] < a->row_bytes)) return AVSG_EINVAL;
        if (a->kv_rows && a->kv_rows[i] > 0x80000000u) return AVSG_EINVAL;
        p.id_limit[i] = a->kv_rows ? a->kv_rows[i] : 0x80000000u;
        cudaPointerAttributes at;
        if (cudaPointerGetAttributes(&at, base) != cudaSuccess) { cudaGetLastError(); return AVSG_EINVAL; }
        if (at.type == cudaMemoryTypeUnregistered || !at.devicePointer) return AVSG_EINVAL;
        p.table_id[i] = i;
        p.verified_len[i] = a->verified_len[i];
        p.kv_base[i] = reinterpret_cast<uint64_t>(at.devicePointer);
        p.kv_stride[i] = a->row_stride ? a->row_stride[i] : a->row_bytes;
    }

    // the array keeps the previous call's contents: status, segment lengths and counters restart at zero
    if (cudaMemsetAsync(sc, 0, offsetof(NoAllocScratch, list), stream) != cudaSuccess) return AVSG_ECUDA;
    if (launch_stage_one(p, a->n, stream) != cudaSuccess) return AVSG_ECUDA;

    XferParams x;
    x.seg = sc->seg; x.miss_list = sc->list; x.status = sc->status;
    x.n_seg = a->n; x.list_stride = list_stride; x.row_bytes = a->row_bytes; x.request_level = 0; x.S = a->buffer_slots;
    if (launch_transfer(x, (uint32_t)g_sm_count[dev], 256, stream) != cudaSuccess) return AVSG_ECUDA;

    if (a->status &&
        cudaMemcpyAsync(a->status, sc->status, sizeof(uint32_t), cudaMemcpyDeviceToDevice, stream) != cudaSuccess)
        return AVSG_ECUDA;
    return AVSG_OK;
}
