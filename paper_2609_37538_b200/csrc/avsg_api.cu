// C ABI of the AVSG decode-step operator (see include/avsg.h): argument
// checking, device state, kernel launches.  No step of the operator runs on
// the host; there is no CPU fallback.
#include <new>
#include <string.h>
#include <vector>

#include <cuda.h>          // types of the one driver entry point fetched at run time (nothing links libcuda)

#include "avsg.h"
#include "avsg_kernels.cuh"

using namespace avsg;

struct avsg_ctx {
    avsg_config cfg;
    uint32_t logS = 0, logH = 0;
    uint32_t s1_cluster = 1;           // blocks that share one table in Stage One (1 = the single-block kernel)
    uint32_t host_status = 0;          // status bits raised on the host side (sticky like the device word)
    uint32_t list_stride = 0;          // entries per miss-list segment
    int sm_count = 0;
    uint32_t xfer_blocks = 0, xfer_threads = 256;
    bool timing = false, events_recorded = false;

    int32_t* d_tok = nullptr;
    int8_t* d_life = nullptr;
    uint8_t* d_buffer = nullptr;
    TableStats* d_stats = nullptr;
    unsigned long long* d_flags = nullptr;         // overlapped Stage Two: per-(table of the call, token) flags
                                                   //   (call number << 32 | miss count) [OVERLAP_MAX_TABLES x TOKENS]
    unsigned long long* d_sync = nullptr;          //   [0] the call number, [1] transfer blocks that are through,
                                                   //   [2] sequence number of the last host-buffer call,
                                                   //   [3] arrivals after a host-buffer call's last token
    S1ParamsBig* big_args = nullptr;               // host: the large Stage One argument block, built in place per call
    unsigned long long* d_trange = nullptr;        // [8] time marks of the last timed call, then [8] their initial values
    unsigned long long* d_trange_init = nullptr;
    int2* d_list = nullptr;
    SegDesc* d_seg = nullptr;
    uint32_t* d_status = nullptr;
    uint16_t* d_where = nullptr;       // direct index, or null
    uint32_t* d_q = nullptr;           // paper-literal mode: packed words, or null
    uint32_t* d_q_snap = nullptr;
    int32_t* d_tok_snap = nullptr;
    int8_t* d_life_snap = nullptr;
    // staging of avsg_step_host
    int32_t* d_idx_stage = nullptr;
    int32_t* d_slots_stage = nullptr;
    uint8_t* d_hit_stage = nullptr;
    int32_t* d_mc_stage = nullptr;
    // copy-engine comparator (pinned host copies of the miss list)
    SegDesc* h_seg = nullptr;
    int2* h_list = nullptr;

    std::vector<uint64_t> kv_host, kv_dev;     // last validated host KV base per table
    std::vector<uint32_t> seen;                // distinctness check of table ids
    uint32_t epoch = 0;
    std::vector<const void*> call_kv_host;     // host pointers of the current call (copy-engine mode)
    std::vector<uint64_t> call_kv_dev;         // their device-visible addresses, resolved before anything is launched
    cudaEvent_t ev[3] = {nullptr, nullptr, nullptr};
    // avsg_step_host: the outputs go back on a side stream while Stage Two runs
    cudaStream_t side = nullptr;
    // cuStreamWaitValue64, when driver and device offer it: in the overlapped mode the output download of a call
    // with host buffers waits for the sequence number Stage One writes once all its outputs exist, instead of for
    // an event between the two grids (which would run them one after the other)
    CUresult (*wait_value64)(CUstream, CUdeviceptr, cuuint64_t, unsigned int) = nullptr;
    unsigned long long host_seq = 0;               // calls with host buffers issued in that mode so far
    cudaEvent_t ev_outputs_ready = nullptr, ev_outputs_copied = nullptr, ev_ids_ready = nullptr;
    uint64_t last_rows = 0;
};

namespace {

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev)
    {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    }
    ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

#define CU(call) do { if ((call) != cudaSuccess) return AVSG_ECUDA; } while (0)

bool is_pow2(uint32_t v) { return v && !(v & (v - 1)); }
uint32_t ilog2(uint32_t v) { uint32_t l = 0; while ((1u << l) < v) ++l; return l; }

void free_all(avsg_ctx* c)
{
    cudaFree(c->d_tok); cudaFree(c->d_life); cudaFree(c->d_buffer); cudaFree(c->d_stats); cudaFree(c->d_trange);
    cudaFree(c->d_flags); cudaFree(c->d_sync);
    delete c->big_args;
    cudaFree(c->d_list); cudaFree(c->d_seg); cudaFree(c->d_status); cudaFree(c->d_where); cudaFree(c->d_q); cudaFree(c->d_q_snap);
    cudaFree(c->d_tok_snap); cudaFree(c->d_life_snap);
    cudaFree(c->d_idx_stage); cudaFree(c->d_slots_stage); cudaFree(c->d_hit_stage); cudaFree(c->d_mc_stage);
    if (c->h_seg) cudaFreeHost(c->h_seg);
    if (c->h_list) cudaFreeHost(c->h_list);
    for (auto& e : c->ev) if (e) cudaEventDestroy(e);
    if (c->ev_outputs_ready) cudaEventDestroy(c->ev_outputs_ready);
    if (c->ev_outputs_copied) cudaEventDestroy(c->ev_outputs_copied);
    if (c->ev_ids_ready) cudaEventDestroy(c->ev_ids_ready);
    if (c->side) cudaStreamDestroy(c->side);
}

int init_tables(avsg_ctx* c, uint32_t first, uint32_t n)
{
    const size_t S = c->cfg.buffer_slots;
    CU(cudaMemset(c->d_tok + first * S, 0xFF, n * S * sizeof(int32_t)));        // id -1: empty
    CU(cudaMemset(c->d_life + first * S, 0xFF, n * S));                         // lifetime -1: dead
    CU(cudaMemset(c->d_buffer + first * S * c->cfg.row_bytes, 0, n * S * c->cfg.row_bytes));
    CU(cudaMemset(c->d_stats + first, 0, n * sizeof(TableStats)));
    if (c->d_q) {                                           // lifetime -1, mapping invalid: 0xFF800000
        std::vector<uint32_t> init(n * S, 0xFF800000u);
        CU(cudaMemcpy(c->d_q + first * S, init.data(), init.size() * sizeof(uint32_t), cudaMemcpyHostToDevice));
    }
    return AVSG_OK;
}

// Device-visible address of a host KV base (pinned + mapped host memory, or device memory).
int resolve_kv(avsg_ctx* c, uint32_t table, const void* host_ptr, uint64_t* dev)
{
    const uint64_t h = reinterpret_cast<uint64_t>(host_ptr);
    if (c->kv_host[table] == h && c->kv_dev[table]) { *dev = c->kv_dev[table]; return AVSG_OK; }
    cudaPointerAttributes at;
    if (cudaPointerGetAttributes(&at, host_ptr) != cudaSuccess) { cudaGetLastError(); return AVSG_EINVAL; }
    if (at.type == cudaMemoryTypeUnregistered || at.devicePointer == nullptr) return AVSG_EINVAL;
    c->kv_host[table] = h;
    c->kv_dev[table] = reinterpret_cast<uint64_t>(at.devicePointer);
    *dev = c->kv_dev[table];
    return AVSG_OK;
}

int check_args(avsg_ctx* c, const avsg_step_args* a)
{
    if (!c || !a) return AVSG_EINVAL;
    if (a->n == 0 || a->n > c->cfg.num_tables || a->n > (uint32_t)XFER_MAX_SEG) return AVSG_EINVAL;
    if (!a->table_ids || !a->indices || !a->kv_base || !(a->verified_len || a->verified_len_dev) || !a->slots)
        return AVSG_EINVAL;
    if (a->n_tokens == 0 || a->n_tokens > c->cfg.max_tokens || a->topk == 0 || a->topk > c->cfg.max_topk)
        return AVSG_EINVAL;
    if ((uint64_t)a->n_tokens * a->topk > c->cfg.buffer_slots) return AVSG_ECAPACITY;      // Eq. 7
    if (++c->epoch == 0) { std::fill(c->seen.begin(), c->seen.end(), 0u); c->epoch = 1; }
    for (uint32_t i = 0; i < a->n; ++i) {
        const uint32_t t = a->table_ids[i];
        if (t >= c->cfg.num_tables || c->seen[t] == c->epoch) return AVSG_EINVAL;
        c->seen[t] = c->epoch;
        if (a->row_stride && (a->row_stride[i] % 16 || a->row_stride[i] < c->cfg.row_bytes)) return AVSG_EINVAL;
        if (!a->kv_base[i] || (reinterpret_cast<uint64_t>(a->kv_base[i]) & 15u)) return AVSG_EINVAL;
        if (a->kv_rows && a->kv_rows[i] > 0x80000000u) return AVSG_EINVAL;
    }
    return AVSG_OK;
}

// Comparator: the miss list goes back to the host, then one asynchronous copy per run of
// consecutive (host row, slot) pairs is queued on the copy engine.
int copy_engine_transfer(avsg_ctx* c, const avsg_step_args* a, cudaStream_t stream)
{
    const uint32_t n = a->n;
    CU(cudaMemcpyAsync(c->h_seg, c->d_seg, n * sizeof(SegDesc), cudaMemcpyDeviceToHost, stream));
    CU(cudaStreamSynchronize(stream));
    uint32_t max_count = 0;
    for (uint32_t i = 0; i < n; ++i) max_count = c->h_seg[i].count > max_count ? c->h_seg[i].count : max_count;
    if (max_count == 0) return AVSG_OK;
    if (max_count > c->list_stride) return AVSG_EDEVICE_STATUS;
    const size_t pitch = (size_t)c->list_stride * sizeof(int2);
    CU(cudaMemcpy2DAsync(c->h_list, pitch, c->d_list, pitch, (size_t)max_count * sizeof(int2), n,
                         cudaMemcpyDeviceToHost, stream));
    CU(cudaStreamSynchronize(stream));
    const uint64_t rb = c->cfg.row_bytes;
    for (uint32_t i = 0; i < n; ++i) {
        const SegDesc& sd = c->h_seg[i];
        const int2* e = c->h_list + (size_t)i * c->list_stride;
        const uint8_t* src_base = static_cast<const uint8_t*>(c->call_kv_host[i]);
        uint32_t k = 0;
        while (k < sd.count) {
            if (e[k].x < 0 || e[k].y < 0 || (uint32_t)e[k].y >= c->cfg.buffer_slots) { ++k; continue; }
            uint32_t run = 1;
            if (sd.src_stride == rb)
                while (k + run < sd.count && e[k + run].x == e[k].x + (int32_t)run && e[k + run].y == e[k].y + (int32_t)run) ++run;
            CU(cudaMemcpyAsync(reinterpret_cast<void*>(sd.dst_base + (uint64_t)e[k].y * rb),
                               src_base + (uint64_t)e[k].x * sd.src_stride, run * rb, cudaMemcpyDefault, stream));
            k += run;
        }
    }
    return AVSG_OK;
}

int step_impl(avsg_ctx* c, const avsg_step_args* a, cudaStream_t stream, bool host_io)
{
    int rc = check_args(c, a);
    if (rc != AVSG_OK) return rc;
    if ((a->stage_one_done || a->arriving) && (host_io || c->cfg.transfer_mode == AVSG_XFER_ALL_K ||
                                               (reinterpret_cast<uint64_t>(a->stage_one_done) & 7u)))
        return AVSG_EINVAL;
    DeviceGuard guard(c->cfg.device);
    if (!guard.ok) return AVSG_ECUDA;

    const uint32_t n = a->n, K = a->topk, n_q = a->n_tokens;
    const size_t n_ids = (size_t)n * n_q * K;
    const int32_t* indices = a->indices;
    int32_t* slots = a->slots;
    uint8_t* hit = a->hit;
    int32_t* miss_count = a->miss_count;
    if (host_io) {
        // The ids go up on the side stream, where they queue behind the previous call's output download (and
        // therefore behind its Stage One, the last reader of the staging buffer) but not behind its Stage Two:
        // when calls are issued back to back the upload hides under the previous call's gather.
        CU(cudaMemcpyAsync(c->d_idx_stage, a->indices, n_ids * sizeof(int32_t), cudaMemcpyHostToDevice, c->side));
        CU(cudaEventRecord(c->ev_ids_ready, c->side));
        CU(cudaStreamWaitEvent(stream, c->ev_ids_ready, 0));
        indices = c->d_idx_stage;
        slots = c->d_slots_stage;
        hit = a->hit ? c->d_hit_stage : nullptr;
        miss_count = a->miss_count ? c->d_mc_stage : nullptr;
    }
    uint32_t mode = c->cfg.transfer_mode;
    // tables per Stage One launch: the small argument block when it is enough (and for the kernels that only have
    // that one), else the large one
    const uint32_t chunk = (n <= (uint32_t)S1_MAX_TABLES || mode == AVSG_XFER_ALL_K || c->cfg.index_mode == AVSG_INDEX_PAPER)
                               ? (uint32_t)S1_MAX_TABLES : (uint32_t)S1_BIG_TABLES;
    if (mode == AVSG_XFER_SM_OVERLAP && (n > chunk || n_q > (uint32_t)OVERLAP_MAX_TOKENS))
        mode = AVSG_XFER_SM_BALANCED;                  // the overlapped kernel pairs with ONE Stage One launch
    // The overlapped transfer grid shares the GPU with the Stage One grid it waits for.  When Stage One's blocks
    // take more than half of the SMs, many transfer blocks only find room once Stage One is over and their fixed
    // shares (Eq. 6) finish late: measured, a 96- or 128-table call with one Stage One block per table is 3-6 %
    // slower overlapped than not (64: 2 % faster).
    // Such calls keep Stage One on S1_ROUND_BLOCKS SMs: its blocks serve the tables round by round and the transfer
    // grid, resident on the other SMs, copies round r's misses while round r + 1 is matched (single-block hash /
    // direct kernels; the cluster and paper-literal kernels run Stage Two after Stage One instead).
    uint32_t round_size = n;
    if (mode == AVSG_XFER_SM_OVERLAP && (uint64_t)n * c->s1_cluster > (uint64_t)c->sm_count / 2) {
        if (c->s1_cluster == 1 && c->cfg.index_mode != AVSG_INDEX_PAPER)
            round_size = S1_ROUND_BLOCKS;
        else
            mode = AVSG_XFER_SM_BALANCED;
    }
    // host buffers in the overlapped mode: no event between the two grids, the download waits for a sequence number
    const bool wait_on_sequence = host_io && mode == AVSG_XFER_SM_OVERLAP && c->wait_value64 != nullptr;
    // the position-level comparator reads the hit mask: use the library's own buffer if the caller wants none
    if (mode == AVSG_XFER_POSITION_LEVEL && !hit) hit = c->d_hit_stage;
    if (c->timing) {
        // grid spans: [0] Stage One first start, [1] its last end, [2], [3] the same for Stage Two
        CU(cudaMemcpyAsync(c->d_trange, c->d_trange_init, 8 * sizeof(unsigned long long), cudaMemcpyDeviceToDevice, stream));
        CU(cudaEventRecord(c->ev[0], stream));
    }

    c->call_kv_host.assign(a->kv_base, a->kv_base + n);
    // every host KV base is resolved (and refused, if the GPU cannot read it) before the first launch of the call:
    // a call either starts completely or not at all
    c->call_kv_dev.resize(n);
    for (uint32_t i = 0; i < n; ++i)
        if ((rc = resolve_kv(c, a->table_ids[i], a->kv_base[i], &c->call_kv_dev[i])) != AVSG_OK) return rc;
    // ids at or beyond this are never looked up or fetched: the table's host rows when the caller states them,
    // and the size of the direct index
    auto id_limit_of = [&](uint32_t i) -> uint32_t {
        uint32_t lim = a->kv_rows ? a->kv_rows[i] : 0x80000000u;
        if (c->d_where && c->cfg.max_context < lim) lim = c->cfg.max_context;
        return lim;
    };
    // Stage One for tables [first, first + cnt) of the call, with the small or the large argument block
    auto stage_one = [&](auto& p, uint32_t first, uint32_t cnt) -> int {
        p.tok = c->d_tok; p.life = c->d_life; p.buffer = c->d_buffer; p.stats = c->d_stats;
        p.miss_list = c->d_list; p.seg = c->d_seg; p.status = c->d_status;
        p.indices = indices; p.slots = slots; p.hit = hit; p.miss_count = miss_count;
        p.S = c->cfg.buffer_slots; p.logH = c->logH; p.row_bytes = c->cfg.row_bytes;
        p.K = K; p.n_q = n_q; p.L = (uint32_t)c->cfg.max_lifetime;
        p.first = first; p.list_stride = c->list_stride;
        p.n_launch = cnt; p.round_size = round_size;
        p.where = c->d_where; p.max_context = c->cfg.max_context;
        p.qword = c->d_q; p.probe_retries = c->cfg.probe_retries; p.hash_a1 = c->cfg.hash_a1; p.hash_a2 = c->cfg.hash_a2;
        p.t_range = c->timing ? c->d_trange : nullptr;
        p.verified_len_dev = a->verified_len_dev;
        // (every field is assigned: the large block is re-used from call to call)
        const bool overlap = mode == AVSG_XFER_SM_OVERLAP;
        p.flags = overlap ? c->d_flags : nullptr;
        p.epoch = reinterpret_cast<const uint32_t*>(c->d_sync);
        // the caller's word: written by Stage One itself, or by the `arriving` kernel behind it when that output
        // is asked for too (the word then also covers it)
        p.done_seq = wait_on_sequence ? c->d_sync + 2
                                      : (a->arriving ? nullptr : reinterpret_cast<unsigned long long*>(a->stage_one_done));
        p.done_ctr = reinterpret_cast<uint32_t*>(c->d_sync + 3);
        p.host_seq = wait_on_sequence ? c->host_seq + 1 : a->stage_one_done_value;
        p.expect = n;
        for (uint32_t i = 0; i < cnt; ++i) {
            p.table_id[i] = a->table_ids[first + i];
            p.verified_len[i] = a->verified_len ? a->verified_len[first + i] : 0;
            p.id_limit[i] = id_limit_of(first + i);
            p.kv_base[i] = c->call_kv_dev[first + i];
            p.kv_stride[i] = a->row_stride ? a->row_stride[first + i] : c->cfg.row_bytes;
        }
        if (c->s1_cluster > 1) CU(launch_stage_one_cluster(p, cnt, c->s1_cluster, stream));
        else CU(launch_stage_one(p, cnt < round_size ? cnt : round_size, stream));
        return AVSG_OK;
    };
    for (uint32_t first = 0; first < n; first += chunk) {
        const uint32_t cnt = n - first < chunk ? n - first : chunk;
        if (mode == AVSG_XFER_ALL_K) {
            AllKParams p;
            p.indices = indices; p.slots = slots; p.hit = hit; p.miss_count = miss_count;
            p.miss_list = c->d_list; p.seg = c->d_seg; p.stats = c->d_stats; p.buffer = c->d_buffer;
            p.status = c->d_status;
            p.S = c->cfg.buffer_slots; p.row_bytes = c->cfg.row_bytes; p.K = K; p.n_q = n_q;
            p.first = first; p.list_stride = c->list_stride;
            for (uint32_t i = 0; i < cnt; ++i) {
                p.table_id[i] = a->table_ids[first + i];
                p.id_limit[i] = id_limit_of(first + i);
                p.kv_base[i] = c->call_kv_dev[first + i];
                p.kv_stride[i] = a->row_stride ? a->row_stride[first + i] : c->cfg.row_bytes;
            }
            CU(launch_all_k_prepare(p, cnt, stream));
        } else if (chunk == (uint32_t)S1_MAX_TABLES) {
            S1Params p;
            if ((rc = stage_one(p, first, cnt)) != AVSG_OK) return rc;
        } else {
            if ((rc = stage_one(*c->big_args, first, cnt)) != AVSG_OK) return rc;
        }
    }
    if (a->arriving) {
        ArrivingParams q;
        q.seg = c->d_seg; q.miss_list = c->d_list; q.slots = slots; q.arriving = a->arriving;
        q.done_seq = reinterpret_cast<unsigned long long*>(a->stage_one_done);
        q.done_ctr = reinterpret_cast<uint32_t*>(c->d_sync + 3);
        q.value = a->stage_one_done_value;
        q.n = n; q.per_table = n_q * K; q.S = c->cfg.buffer_slots; q.list_stride = c->list_stride;
        q.flags = mode == AVSG_XFER_SM_OVERLAP ? c->d_flags : nullptr;
        q.epoch = reinterpret_cast<const uint32_t*>(c->d_sync);
        q.n_q = n_q; q.status = c->d_status;
        CU(launch_arriving(q, (uint32_t)c->sm_count, stream));
    }
    // (no event between the two grids in overlap mode: it would serialise them; ev[1] is recorded with ev[2])
    if (c->timing && mode != AVSG_XFER_SM_OVERLAP) CU(cudaEventRecord(c->ev[1], stream));

    // The slot table, hit mask and miss counts are final once Stage One has run.  They travel device -> host on a
    // side stream while Stage Two pulls rows host -> device: the two directions of the link overlap.
    auto download_outputs = [&]() -> int {
        CU(cudaMemcpyAsync(a->slots, c->d_slots_stage, n_ids * sizeof(int32_t), cudaMemcpyDeviceToHost, c->side));
        if (a->hit) CU(cudaMemcpyAsync(a->hit, c->d_hit_stage, n_ids, cudaMemcpyDeviceToHost, c->side));
        if (a->miss_count)
            CU(cudaMemcpyAsync(a->miss_count, c->d_mc_stage, (size_t)n * n_q * sizeof(int32_t), cudaMemcpyDeviceToHost, c->side));
        CU(cudaEventRecord(c->ev_outputs_copied, c->side));
        return AVSG_OK;
    };
    if (host_io && !wait_on_sequence) {
        CU(cudaEventRecord(c->ev_outputs_ready, stream));
        CU(cudaStreamWaitEvent(c->side, c->ev_outputs_ready, 0));
        if ((rc = download_outputs()) != AVSG_OK) return rc;
    }

    if (mode == AVSG_XFER_COPY_ENGINE) {
        if ((rc = copy_engine_transfer(c, a, stream)) != AVSG_OK) return rc;
    } else if (mode == AVSG_XFER_POSITION_LEVEL) {
        PosParams q;
        q.seg = c->d_seg; q.indices = indices; q.slots = slots; q.hit = hit; q.status = c->d_status;
        q.n = n; q.per_table = n_q * K; q.row_bytes = c->cfg.row_bytes; q.S = c->cfg.buffer_slots;
        CU(launch_transfer_positions(q, c->xfer_blocks ? c->xfer_blocks : (uint32_t)c->sm_count, c->xfer_threads, stream));
    } else if (mode == AVSG_XFER_SM_OVERLAP) {
        XferOverlapParams x;
        x.seg = c->d_seg; x.miss_list = c->d_list; x.status = c->d_status;
        x.flags = c->d_flags; x.epoch = reinterpret_cast<uint32_t*>(c->d_sync);
        x.done = reinterpret_cast<uint32_t*>(c->d_sync + 1);
        x.n = n; x.n_q = n_q; x.list_stride = c->list_stride; x.row_bytes = c->cfg.row_bytes; x.S = c->cfg.buffer_slots;
        x.round_size = round_size; x.expect_extra = 0;
        x.t_range = c->timing ? c->d_trange + 2 : nullptr;
        if (launch_transfer_overlap(x, c->xfer_blocks ? c->xfer_blocks : (uint32_t)c->sm_count, c->xfer_threads, stream)
            != cudaSuccess) {
            // Stage One has run and written flags with the current call number, which nothing will advance: wipe
            // them here, in stream order, and remember that this call reserved slots whose rows were never copied
            cudaGetLastError();
            cudaMemsetAsync(c->d_flags, 0, (size_t)OVERLAP_MAX_TABLES * OVERLAP_MAX_TOKENS * sizeof(unsigned long long), stream);
            c->host_status |= AVSG_STATUS_LAUNCH_FAILED;
            return AVSG_ECUDA;
        }
        if (wait_on_sequence) {
            c->host_seq += 1;
            if (c->wait_value64(c->side, reinterpret_cast<CUdeviceptr>(c->d_sync + 2), c->host_seq,
                                CU_STREAM_WAIT_VALUE_GEQ) != CUDA_SUCCESS)
                return AVSG_ECUDA;
            if ((rc = download_outputs()) != AVSG_OK) return rc;
        }
    } else {
        XferParams x;
        x.seg = c->d_seg; x.miss_list = c->d_list; x.status = c->d_status;
        x.n_seg = n; x.list_stride = c->list_stride; x.row_bytes = c->cfg.row_bytes;
        x.request_level = mode == AVSG_XFER_REQUEST_LEVEL; x.S = c->cfg.buffer_slots;
        x.t_range = c->timing ? c->d_trange + 2 : nullptr;
        const uint32_t blocks = x.request_level ? n : (c->xfer_blocks ? c->xfer_blocks : (uint32_t)c->sm_count);
        if (launch_transfer(x, blocks, c->xfer_threads, stream) != cudaSuccess) {
            cudaGetLastError();
            c->host_status |= AVSG_STATUS_LAUNCH_FAILED;
            return AVSG_ECUDA;
        }
    }
    if (c->timing) {
        if (mode == AVSG_XFER_SM_OVERLAP) CU(cudaEventRecord(c->ev[1], stream));
        CU(cudaEventRecord(c->ev[2], stream));
        c->events_recorded = true;
    }

    if (host_io) CU(cudaStreamWaitEvent(stream, c->ev_outputs_copied, 0));     // the call ends when the outputs are home
    return AVSG_OK;
}

int read_status(avsg_ctx* c, uint32_t* word)
{
    uint32_t st = 0;
    CU(cudaMemcpy(&st, c->d_status, sizeof(st), cudaMemcpyDeviceToHost));
    st |= c->host_status;
    if (word) *word = st;
    return st ? AVSG_EDEVICE_STATUS : AVSG_OK;
}

}  // namespace

extern "C" {

int avsg_create(const avsg_config* cfg, avsg_ctx** out)
{
    if (!cfg || !out) return AVSG_EINVAL;
    if (cfg->num_tables == 0 || !is_pow2(cfg->buffer_slots) || cfg->buffer_slots < 32) return AVSG_EINVAL;
    if (cfg->buffer_slots > 32768) return AVSG_EUNSUPPORTED;
    if (cfg->stage_one_cluster > 8 || (cfg->stage_one_cluster & (cfg->stage_one_cluster - 1))) return AVSG_EINVAL;
    if (cfg->max_topk > 32768) return AVSG_EUNSUPPORTED;
    if (cfg->row_bytes == 0 || cfg->row_bytes % 16) return AVSG_EINVAL;
    if (cfg->max_topk == 0 || cfg->max_tokens == 0) return AVSG_EINVAL;
    if (cfg->max_lifetime < 1 || cfg->max_lifetime > 126) return AVSG_EINVAL;
    if (cfg->transfer_mode > AVSG_XFER_SM_OVERLAP || cfg->index_mode > AVSG_INDEX_PAPER) return AVSG_EINVAL;
    if (cfg->index_mode == AVSG_INDEX_DIRECT && cfg->max_context == 0) return AVSG_EINVAL;
    if ((uint64_t)cfg->max_topk * cfg->max_tokens > cfg->buffer_slots) return AVSG_ECAPACITY;   // Eq. 7
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || cfg->device < 0 || cfg->device >= ndev) return AVSG_ECUDA;
    DeviceGuard guard(cfg->device);
    if (!guard.ok) return AVSG_ECUDA;

    avsg_ctx* c = new (std::nothrow) avsg_ctx();
    if (!c) return AVSG_ENOMEM;
    c->cfg = *cfg;
    if (c->cfg.probe_retries == 0) c->cfg.probe_retries = 3;
    if (c->cfg.hash_a1 == 0) c->cfg.hash_a1 = 1000003u;
    if (c->cfg.hash_a2 == 0) c->cfg.hash_a2 = 998244353u;
    c->logS = ilog2(cfg->buffer_slots);
    c->logH = c->logS + 1;
    c->list_stride = cfg->max_topk * cfg->max_tokens;
    const size_t T = cfg->num_tables, S = cfg->buffer_slots;
    c->kv_host.assign(T, 0); c->kv_dev.assign(T, 0); c->seen.assign(T, 0);

    int max_smem = 0;
    cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, cfg->device);
    cudaDeviceGetAttribute(&max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, cfg->device);
    // Blocks per table in Stage One: what the configuration asks for, else the single-block kernel while the table
    // fits one SM's shared memory and the smallest cluster that holds it above that.
    {
        const bool direct = cfg->index_mode == AVSG_INDEX_DIRECT;
        const uint32_t S = cfg->buffer_slots, K = cfg->max_topk, L = (uint32_t)cfg->max_lifetime;
        auto fits = [&](uint32_t C) -> bool {
            if (cfg->index_mode == AVSG_INDEX_PAPER)
                return C == 1 && S <= 8192 && stage_one_paper_smem_bytes(S, K, L) <= (size_t)max_smem;
            if (C == 1) return S <= 8192 && stage_one_smem_bytes(S, K, L, direct) <= (size_t)max_smem;
            return S / C >= 32 && S / C <= 8192 && stage_one_cluster_smem_bytes(S, K, L, C, direct) <= (size_t)max_smem;
        };
        uint32_t C = cfg->stage_one_cluster;
        if (C == 0)
            for (C = 1; C <= 8 && !fits(C); C *= 2) {}
        if (C > 8 || !fits(C)) { delete c; return AVSG_EUNSUPPORTED; }
        c->s1_cluster = C;
    }
    // always raise the kernels' dynamic shared-memory limit to the device maximum: the attribute is
    // per function, so a context with a small table must not lower it under a context with a large one
    if (stage_one_prepare((size_t)max_smem) != cudaSuccess || stage_one_cluster_prepare((size_t)max_smem) != cudaSuccess ||
        transfer_prepare() != cudaSuccess || arriving_prepare() != cudaSuccess) {
        delete c; return AVSG_ECUDA;
    }
    // a cluster shape that fits on paper may still find no home on the device (blocks of one cluster share a GPC)
    if (c->s1_cluster > 1 &&
        stage_one_cluster_max_active(cfg->buffer_slots, cfg->max_topk, (uint32_t)cfg->max_lifetime, c->s1_cluster,
                                     cfg->index_mode == AVSG_INDEX_DIRECT) < 1) {
        delete c; return AVSG_EUNSUPPORTED;
    }

    const size_t n_ids = T * c->list_stride;
    bool ok = true;
    ok = ok && cudaMalloc(&c->d_tok, T * S * sizeof(int32_t)) == cudaSuccess;
    ok = ok && cudaMalloc(&c->d_life, T * S) == cudaSuccess;
    ok = ok && cudaMalloc(&c->d_buffer, T * S * cfg->row_bytes) == cudaSuccess;
    ok = ok && cudaMalloc(&c->d_stats, T * sizeof(TableStats)) == cudaSuccess;
    ok = ok && cudaMalloc(&c->d_trange, 16 * sizeof(unsigned long long)) == cudaSuccess;
    ok = ok && cudaMalloc(&c->d_flags, (size_t)OVERLAP_MAX_TABLES * OVERLAP_MAX_TOKENS * sizeof(unsigned long long)) == cudaSuccess;
    ok = ok && cudaMalloc(&c->d_sync, 8 * sizeof(unsigned long long)) == cudaSuccess;
    c->big_args = new (std::nothrow) S1ParamsBig();
    ok = ok && c->big_args != nullptr;
    ok = ok && cudaMalloc(&c->d_list, n_ids * sizeof(int2)) == cudaSuccess;
    ok = ok && cudaMalloc(&c->d_seg, T * sizeof(SegDesc)) == cudaSuccess;
    ok = ok && cudaMalloc(&c->d_status, 256) == cudaSuccess;
    if (cfg->index_mode == AVSG_INDEX_PAPER) {
        ok = ok && cudaMalloc(&c->d_q, T * S * sizeof(uint32_t)) == cudaSuccess;
        ok = ok && cudaMalloc(&c->d_q_snap, T * S * sizeof(uint32_t)) == cudaSuccess;
    }
    if (cfg->index_mode == AVSG_INDEX_DIRECT)
        ok = ok && cudaMalloc(&c->d_where, T * (size_t)cfg->max_context * sizeof(uint16_t)) == cudaSuccess;
    ok = ok && cudaMalloc(&c->d_tok_snap, T * S * sizeof(int32_t)) == cudaSuccess;
    ok = ok && cudaMalloc(&c->d_life_snap, T * S) == cudaSuccess;
    ok = ok && cudaMalloc(&c->d_idx_stage, n_ids * sizeof(int32_t)) == cudaSuccess;
    ok = ok && cudaMalloc(&c->d_slots_stage, n_ids * sizeof(int32_t)) == cudaSuccess;
    ok = ok && cudaMalloc(&c->d_hit_stage, n_ids) == cudaSuccess;
    ok = ok && cudaMalloc(&c->d_mc_stage, T * cfg->max_tokens * sizeof(int32_t)) == cudaSuccess;
    ok = ok && cudaHostAlloc(&c->h_seg, T * sizeof(SegDesc), cudaHostAllocDefault) == cudaSuccess;
    ok = ok && cudaHostAlloc(&c->h_list, n_ids * sizeof(int2), cudaHostAllocDefault) == cudaSuccess;
    for (auto& e : c->ev) ok = ok && cudaEventCreate(&e) == cudaSuccess;
    ok = ok && cudaStreamCreateWithFlags(&c->side, cudaStreamNonBlocking) == cudaSuccess;
    {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult found = cudaDriverEntryPointSymbolNotFound;
        int can64 = 0;
        // attribute 122 of the driver's numbering (the runtime's enum does not name it): 64-bit stream memory operations
        if (cudaGetDriverEntryPoint("cuStreamWaitValue64", &fn, cudaEnableDefault, &found) == cudaSuccess &&
            found == cudaDriverEntryPointSuccess &&
            cudaDeviceGetAttribute(&can64, static_cast<cudaDeviceAttr>(CU_DEVICE_ATTRIBUTE_CAN_USE_64_BIT_STREAM_MEM_OPS),
                                   cfg->device) == cudaSuccess && can64)
            c->wait_value64 = reinterpret_cast<CUresult (*)(CUstream, CUdeviceptr, cuuint64_t, unsigned int)>(fn);
        else
            cudaGetLastError();
    }
    ok = ok && cudaEventCreateWithFlags(&c->ev_outputs_ready, cudaEventDisableTiming) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&c->ev_outputs_copied, cudaEventDisableTiming) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&c->ev_ids_ready, cudaEventDisableTiming) == cudaSuccess;
    if (!ok) { cudaGetLastError(); free_all(c); delete c; return AVSG_ENOMEM; }
    {
        // [0] Stage One first start, [1] its last end; Stage Two: [2] first start, [3] last end, [4] first copy loop,
        // [5] first row in, [6] first block done; minima start at "never", maxima at 0
        const unsigned long long never = ~0ull, first_epoch = 1;      // call numbers start at 1: a zeroed flag is never valid
        const unsigned long long init[16] = {never, 0, never, 0, never, never, never, 0, never, 0, never, 0, never, never, never, 0};
        c->d_trange_init = c->d_trange + 8;
        if (cudaMemcpy(c->d_trange, init, sizeof(init), cudaMemcpyHostToDevice) != cudaSuccess ||
            cudaMemset(c->d_flags, 0, (size_t)OVERLAP_MAX_TABLES * OVERLAP_MAX_TOKENS * sizeof(unsigned long long)) != cudaSuccess ||
            cudaMemset(c->d_sync, 0, 8 * sizeof(unsigned long long)) != cudaSuccess ||
            cudaMemcpy(c->d_sync, &first_epoch, sizeof(first_epoch), cudaMemcpyHostToDevice) != cudaSuccess) {
            free_all(c); delete c; return AVSG_ECUDA;
        }
    }
    if ((c->d_where && cudaMemset(c->d_where, 0xFF, T * (size_t)cfg->max_context * sizeof(uint16_t)) != cudaSuccess) ||
        cudaMemset(c->d_status, 0, 256) != cudaSuccess || cudaMemset(c->d_seg, 0, T * sizeof(SegDesc)) != cudaSuccess ||
        init_tables(c, 0, (uint32_t)T) != AVSG_OK || cudaDeviceSynchronize() != cudaSuccess) {
        free_all(c); delete c; return AVSG_ECUDA;
    }
    *out = c;
    return AVSG_OK;
}

int avsg_destroy(avsg_ctx* c)
{
    if (!c) return AVSG_EINVAL;
    DeviceGuard guard(c->cfg.device);
    cudaDeviceSynchronize();
    free_all(c);
    delete c;
    return AVSG_OK;
}

int avsg_reset(avsg_ctx* c, const uint32_t* table_ids, uint32_t n)
{
    if (!c || (!table_ids && n)) return AVSG_EINVAL;
    for (uint32_t i = 0; i < n; ++i) if (table_ids[i] >= c->cfg.num_tables) return AVSG_EINVAL;
    DeviceGuard guard(c->cfg.device);
    if (!guard.ok) return AVSG_ECUDA;
    CU(cudaDeviceSynchronize());
    for (uint32_t i = 0; i < n; ++i) {
        int rc = init_tables(c, table_ids[i], 1);
        if (rc != AVSG_OK) return rc;
        c->kv_host[table_ids[i]] = 0; c->kv_dev[table_ids[i]] = 0;
    }
    CU(cudaDeviceSynchronize());
    return AVSG_OK;
}

int avsg_reset_async(avsg_ctx* c, const uint32_t* table_ids, uint32_t n, void* cuda_stream)
{
    if (!c || (!table_ids && n)) return AVSG_EINVAL;
    for (uint32_t i = 0; i < n; ++i) if (table_ids[i] >= c->cfg.num_tables) return AVSG_EINVAL;
    DeviceGuard guard(c->cfg.device);
    if (!guard.ok) return AVSG_ECUDA;
    for (uint32_t first = 0; first < n; first += S1_MAX_TABLES) {
        const uint32_t cnt = n - first < (uint32_t)S1_MAX_TABLES ? n - first : (uint32_t)S1_MAX_TABLES;
        ResetParams p;
        p.tok = c->d_tok; p.life = c->d_life; p.buffer = c->d_buffer; p.stats = c->d_stats; p.qword = c->d_q;
        p.S = c->cfg.buffer_slots; p.row_bytes = c->cfg.row_bytes;
        for (uint32_t i = 0; i < cnt; ++i) {
            p.table_id[i] = table_ids[first + i];
            c->kv_host[p.table_id[i]] = 0; c->kv_dev[p.table_id[i]] = 0;      // the next request brings its own host KV
        }
        CU(launch_reset_tables(p, cnt, static_cast<cudaStream_t>(cuda_stream)));
    }
    return AVSG_OK;
}

int avsg_step(avsg_ctx* c, const avsg_step_args* a, void* stream)
{
    return step_impl(c, a, static_cast<cudaStream_t>(stream), false);
}

int avsg_step_host(avsg_ctx* c, const avsg_step_args* a, void* stream)
{
    return step_impl(c, a, static_cast<cudaStream_t>(stream), true);
}

int avsg_buffer(avsg_ctx* c, uint32_t table_id, void** d_rows)
{
    if (!c || !d_rows || table_id >= c->cfg.num_tables) return AVSG_EINVAL;
    *d_rows = c->d_buffer + (size_t)table_id * c->cfg.buffer_slots * c->cfg.row_bytes;
    return AVSG_OK;
}

int avsg_stats(avsg_ctx* c, avsg_stats_t* out)
{
    if (!c || !out) return AVSG_EINVAL;
    DeviceGuard guard(c->cfg.device);
    if (!guard.ok) return AVSG_ECUDA;
    CU(cudaDeviceSynchronize());
    std::vector<TableStats> h(c->cfg.num_tables);
    CU(cudaMemcpy(h.data(), c->d_stats, h.size() * sizeof(TableStats), cudaMemcpyDeviceToHost));
    memset(out, 0, sizeof(*out));
    for (const TableStats& t : h) {
        out->steps += t.steps; out->tokens += t.tokens; out->hits += t.hits; out->misses += t.misses;
        out->rows_copied += t.rows; out->extra_decays += t.extra_decays;
    }
    out->bytes_copied = out->rows_copied * c->cfg.row_bytes;
    if (c->timing && c->events_recorded) {
        float a = 0.f, b = 0.f;
        if (cudaEventElapsedTime(&a, c->ev[0], c->ev[1]) == cudaSuccess) out->last_stage_one_us = a * 1000.f;
        if (cudaEventElapsedTime(&b, c->ev[1], c->ev[2]) == cudaSuccess) out->last_transfer_us = b * 1000.f;
        cudaGetLastError();
        unsigned long long r[8];
        CU(cudaMemcpy(r, c->d_trange, sizeof(r), cudaMemcpyDeviceToHost));
        if (r[1] > r[0]) out->last_stage_one_kernel_us = (float)(r[1] - r[0]) * 1e-3f;
        if (r[3] > r[2]) out->last_transfer_kernel_us = (float)(r[3] - r[2]) * 1e-3f;
        if (r[3] > r[2] && r[1] > r[0] && r[2] >= r[0]) out->last_transfer_start_us = (float)(r[2] - r[0]) * 1e-3f;
        const unsigned long long never = ~0ull;
        if (r[1] > r[0] && r[3] > r[2]) {                 // the other marks, all measured from Stage One's first start
            if (r[4] != never && r[4] >= r[0]) out->last_copy_start_us = (float)(r[4] - r[0]) * 1e-3f;
            if (r[5] != never && r[5] >= r[0]) out->last_first_row_us = (float)(r[5] - r[0]) * 1e-3f;
            if (r[6] != never && r[6] >= r[0]) out->last_first_block_done_us = (float)(r[6] - r[0]) * 1e-3f;
            if (r[3] >= r[0]) out->last_call_kernel_us = (float)((r[3] > r[1] ? r[3] : r[1]) - r[0]) * 1e-3f;
        }
    }
    out->last_rows = out->rows_copied - c->last_rows;
    c->last_rows = out->rows_copied;
    return read_status(c, nullptr);
}

int avsg_table_stats(avsg_ctx* c, uint32_t table_id, avsg_stats_t* out)
{
    if (!c || !out || table_id >= c->cfg.num_tables) return AVSG_EINVAL;
    DeviceGuard guard(c->cfg.device);
    if (!guard.ok) return AVSG_ECUDA;
    CU(cudaDeviceSynchronize());
    TableStats t;
    CU(cudaMemcpy(&t, c->d_stats + table_id, sizeof(t), cudaMemcpyDeviceToHost));
    memset(out, 0, sizeof(*out));
    out->steps = t.steps; out->tokens = t.tokens; out->hits = t.hits; out->misses = t.misses;
    out->rows_copied = t.rows; out->extra_decays = t.extra_decays;
    out->bytes_copied = out->rows_copied * c->cfg.row_bytes;
    return read_status(c, nullptr);
}

int avsg_sync_status(avsg_ctx* c, uint32_t* status_word)
{
    if (!c) return AVSG_EINVAL;
    DeviceGuard guard(c->cfg.device);
    if (!guard.ok) return AVSG_ECUDA;
    CU(cudaDeviceSynchronize());
    return read_status(c, status_word);
}

int avsg_clear_status(avsg_ctx* c)
{
    if (!c) return AVSG_EINVAL;
    DeviceGuard guard(c->cfg.device);
    if (!guard.ok) return AVSG_ECUDA;
    CU(cudaDeviceSynchronize());
    CU(cudaMemset(c->d_status, 0, sizeof(uint32_t)));
    // a transfer kernel that gave up may have left the per-token counters of the overlapped mode raised
    // (the flags of the overlapped mode carry their call's number and need no clearing; the two arrival counters
    // wrap to zero by themselves unless a grid was lost half way)
    CU(cudaMemset(c->d_sync + 1, 0, sizeof(unsigned long long)));
    CU(cudaMemset(c->d_sync + 3, 0, sizeof(unsigned long long)));
    c->host_status = 0;
    return AVSG_OK;
}

int avsg_probe_wait_limit(avsg_ctx* c, void* cuda_stream)
{
    if (!c) return AVSG_EINVAL;
    DeviceGuard guard(c->cfg.device);
    if (!guard.ok) return AVSG_ECUDA;
    XferOverlapParams x;
    x.seg = c->d_seg; x.miss_list = c->d_list; x.status = c->d_status;
    x.flags = c->d_flags; x.epoch = reinterpret_cast<uint32_t*>(c->d_sync);
    x.done = reinterpret_cast<uint32_t*>(c->d_sync + 1);
    x.n = 1; x.n_q = 1; x.list_stride = c->list_stride; x.row_bytes = c->cfg.row_bytes; x.S = c->cfg.buffer_slots;
    x.round_size = 1; x.expect_extra = 0x40000000u;     // a call number no Stage One will ever write: the wait must run out
    CU(launch_transfer_overlap(x, c->xfer_blocks ? c->xfer_blocks : (uint32_t)c->sm_count, c->xfer_threads,
                               static_cast<cudaStream_t>(cuda_stream)));
    return AVSG_OK;
}

int avsg_export_state(avsg_ctx* c, uint32_t table_id, int32_t* tok, int8_t* life)
{
    if (!c || !tok || !life || table_id >= c->cfg.num_tables) return AVSG_EINVAL;
    DeviceGuard guard(c->cfg.device);
    if (!guard.ok) return AVSG_ECUDA;
    const size_t S = c->cfg.buffer_slots;
    CU(cudaDeviceSynchronize());
    CU(cudaMemcpy(tok, c->d_tok + table_id * S, S * sizeof(int32_t), cudaMemcpyDeviceToHost));
    CU(cudaMemcpy(life, c->d_life + table_id * S, S, cudaMemcpyDeviceToHost));
    return read_status(c, nullptr);
}

int avsg_import_state(avsg_ctx* c, uint32_t table_id, const int32_t* tok, const int8_t* life)
{
    if (!c || !tok || !life || table_id >= c->cfg.num_tables) return AVSG_EINVAL;
    const size_t S = c->cfg.buffer_slots;
    for (size_t j = 0; j < S; ++j)
        if (life[j] < -1 || life[j] > c->cfg.max_lifetime || tok[j] < -1) return AVSG_EINVAL;
    DeviceGuard guard(c->cfg.device);
    if (!guard.ok) return AVSG_ECUDA;
    CU(cudaDeviceSynchronize());
    CU(cudaMemcpy(c->d_tok + table_id * S, tok, S * sizeof(int32_t), cudaMemcpyHostToDevice));
    CU(cudaMemcpy(c->d_life + table_id * S, life, S, cudaMemcpyHostToDevice));
    if (c->d_where) {
        CU(launch_direct_index_from_state(c->d_tok, c->d_where, table_id, 1, c->cfg.buffer_slots, c->cfg.max_context, nullptr));
        CU(cudaDeviceSynchronize());
    }
    if (c->d_q) {                                           // ids and lifetimes kept, every mapping invalid
        std::vector<uint32_t> q(S);
        for (size_t j = 0; j < S; ++j) q[j] = ((uint32_t)(uint8_t)life[j] << 24) | 0x00800000u;
        CU(cudaMemcpy(c->d_q + table_id * S, q.data(), S * sizeof(uint32_t), cudaMemcpyHostToDevice));
    }
    return AVSG_OK;
}

int avsg_export_hash_state(avsg_ctx* c, uint32_t table_id, int32_t* cc, uint32_t* q)
{
    if (!c || !cc || !q || table_id >= c->cfg.num_tables || !c->d_q) return AVSG_EINVAL;
    DeviceGuard guard(c->cfg.device);
    if (!guard.ok) return AVSG_ECUDA;
    const size_t S = c->cfg.buffer_slots;
    CU(cudaDeviceSynchronize());
    CU(cudaMemcpy(cc, c->d_tok + table_id * S, S * sizeof(int32_t), cudaMemcpyDeviceToHost));
    CU(cudaMemcpy(q, c->d_q + table_id * S, S * sizeof(uint32_t), cudaMemcpyDeviceToHost));
    return read_status(c, nullptr);
}

int avsg_import_hash_state(avsg_ctx* c, uint32_t table_id, const int32_t* cc, const uint32_t* q)
{
    if (!c || !cc || !q || table_id >= c->cfg.num_tables || !c->d_q) return AVSG_EINVAL;
    const size_t S = c->cfg.buffer_slots;
    std::vector<int8_t> life(S);
    for (size_t j = 0; j < S; ++j) {
        life[j] = (int8_t)(q[j] >> 24);
        if (life[j] < -1 || life[j] > c->cfg.max_lifetime || cc[j] < -1) return AVSG_EINVAL;
    }
    DeviceGuard guard(c->cfg.device);
    if (!guard.ok) return AVSG_ECUDA;
    CU(cudaDeviceSynchronize());
    CU(cudaMemcpy(c->d_tok + table_id * S, cc, S * sizeof(int32_t), cudaMemcpyHostToDevice));
    CU(cudaMemcpy(c->d_q + table_id * S, q, S * sizeof(uint32_t), cudaMemcpyHostToDevice));
    CU(cudaMemcpy(c->d_life + table_id * S, life.data(), S, cudaMemcpyHostToDevice));
    return AVSG_OK;
}

int avsg_save_state(avsg_ctx* c, void* stream)
{
    if (!c) return AVSG_EINVAL;
    DeviceGuard guard(c->cfg.device);
    if (!guard.ok) return AVSG_ECUDA;
    const size_t n = (size_t)c->cfg.num_tables * c->cfg.buffer_slots;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    CU(cudaMemcpyAsync(c->d_tok_snap, c->d_tok, n * sizeof(int32_t), cudaMemcpyDeviceToDevice, s));
    CU(cudaMemcpyAsync(c->d_life_snap, c->d_life, n, cudaMemcpyDeviceToDevice, s));
    if (c->d_q) CU(cudaMemcpyAsync(c->d_q_snap, c->d_q, n * sizeof(uint32_t), cudaMemcpyDeviceToDevice, s));
    return AVSG_OK;
}

int avsg_restore_state(avsg_ctx* c, void* stream)
{
    if (!c) return AVSG_EINVAL;
    DeviceGuard guard(c->cfg.device);
    if (!guard.ok) return AVSG_ECUDA;
    const size_t n = (size_t)c->cfg.num_tables * c->cfg.buffer_slots;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    CU(cudaMemcpyAsync(c->d_tok, c->d_tok_snap, n * sizeof(int32_t), cudaMemcpyDeviceToDevice, s));
    CU(cudaMemcpyAsync(c->d_life, c->d_life_snap, n, cudaMemcpyDeviceToDevice, s));
    if (c->d_q) CU(cudaMemcpyAsync(c->d_q, c->d_q_snap, n * sizeof(uint32_t), cudaMemcpyDeviceToDevice, s));
    if (c->d_where)
        CU(launch_direct_index_from_state(c->d_tok, c->d_where, 0, c->cfg.num_tables, c->cfg.buffer_slots,
                                          c->cfg.max_context, s));
    return AVSG_OK;
}

int avsg_set_transfer_mode(avsg_ctx* c, uint32_t mode)
{
    if (!c || mode > AVSG_XFER_SM_OVERLAP) return AVSG_EINVAL;
    c->cfg.transfer_mode = mode;
    return AVSG_OK;
}

int avsg_set_timing(avsg_ctx* c, int enable)
{
    if (!c) return AVSG_EINVAL;
    c->timing = enable != 0;
    c->events_recorded = false;
    return AVSG_OK;
}

int avsg_set_transfer_geometry(avsg_ctx* c, uint32_t blocks, uint32_t threads)
{
    if (!c || threads < 32 || threads > 1024 || threads % 32 || blocks > 65535) return AVSG_EINVAL;
    c->xfer_blocks = blocks;
    c->xfer_threads = threads;
    return AVSG_OK;
}

const char* avsg_strerror(int code)
{
    switch (code) {
        case AVSG_OK: return "ok";
        case AVSG_EINVAL: return "invalid argument";
        case AVSG_ENOMEM: return "out of memory";
        case AVSG_ECUDA: return "CUDA runtime error";
        case AVSG_ECAPACITY: return "buffer_slots < n_tokens * topk (capacity bound violated)";
        case AVSG_EDEVICE_STATUS: return "a kernel reported a problem in the device status word";
        case AVSG_EUNSUPPORTED: return "shape not supported by this build";
        default: return "unknown error";
    }
}

}  // extern "C"
