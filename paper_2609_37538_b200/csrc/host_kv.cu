// Host KV pool memory: page-locked, device-mapped ranges for a table's host
// KV, optionally backed by transparent 2 MiB pages (App. G keeps the host KV
// pool in an mmap of huge pages).  Host code only; no kernel lives here.
//
// Why the page size matters to the gather: every missed row is read by the
// SMs straight from this memory, and a steady call touches a few thousand
// rows spread over gigabytes.  With 4 KiB pages nearly every row sits on a
// page of its own; with 2 MiB pages the same rows share far fewer
// translations on the way through the host bridge.
#include <cuda_runtime.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>
#include <sys/mman.h>

#include <map>
#include <mutex>

#include "avsg.h"

namespace {

constexpr size_t HUGE_PAGE = size_t(2) << 20;

struct Range {
    void*  map_base;   // what mmap returned
    size_t map_bytes;  // what munmap takes
    size_t bytes;      // registered length, a multiple of HUGE_PAGE
};

std::mutex g_ranges_mutex;
std::map<void*, Range> g_ranges;

// Sums the AnonHugePages figures of the mappings inside [lo, hi) as the kernel
// lists them for this process.  0 when the list cannot be read.
uint64_t huge_bytes_in(uintptr_t lo, uintptr_t hi)
{
    FILE* f = fopen("/proc/self/smaps", "r");
    if (!f) return 0;
    char line[512];
    bool inside = false;
    uint64_t total = 0;
    while (fgets(line, sizeof line, f)) {
        unsigned long long a = 0, b = 0;
        int consumed = 0;
        if (sscanf(line, "%llx-%llx %n", &a, &b, &consumed) == 2 && consumed > 0 && line[consumed - 1] == ' ') {
            inside = (uintptr_t)a >= lo && (uintptr_t)b <= hi;
            continue;
        }
        unsigned long long kb = 0;
        if (inside && sscanf(line, "AnonHugePages: %llu kB", &kb) == 1) total += (uint64_t)kb << 10;
    }
    fclose(f);
    return total;
}

}  // namespace

extern "C" {

int avsg_host_kv_alloc(size_t bytes, uint32_t flags, void** out, uint64_t* huge_bytes)
{
    if (!out || bytes == 0 || (flags & ~AVSG_HOST_KV_HUGE_PAGES)) return AVSG_EINVAL;
    *out = nullptr;
    if (huge_bytes) *huge_bytes = 0;
    if (bytes > (size_t(1) << 46)) return AVSG_EINVAL;
    const size_t len = (bytes + HUGE_PAGE - 1) / HUGE_PAGE * HUGE_PAGE;
    const size_t map_bytes = len + HUGE_PAGE;                       // room to align the start
    void* map_base = mmap(nullptr, map_bytes, PROT_READ | PROT_WRITE, MAP_PRIVATE | MAP_ANONYMOUS, -1, 0);
    if (map_base == MAP_FAILED) return AVSG_ENOMEM;
    const uintptr_t start = ((uintptr_t)map_base + HUGE_PAGE - 1) / HUGE_PAGE * HUGE_PAGE;
    void* base = (void*)start;
    if (flags & AVSG_HOST_KV_HUGE_PAGES) (void)madvise(base, len, MADV_HUGEPAGE);   // advisory
    memset(base, 0, len);                                           // first touch, by this thread
    if (cudaHostRegister(base, len, cudaHostRegisterPortable | cudaHostRegisterMapped) != cudaSuccess) {
        (void)cudaGetLastError();
        munmap(map_base, map_bytes);
        return AVSG_ECUDA;
    }
    if (huge_bytes) *huge_bytes = huge_bytes_in(start, start + len);
    {
        std::lock_guard<std::mutex> lock(g_ranges_mutex);
        g_ranges[base] = Range{map_base, map_bytes, len};
    }
    *out = base;
    return AVSG_OK;
}

int avsg_host_kv_free(void* base)
{
    if (!base) return AVSG_EINVAL;
    Range r;
    {
        std::lock_guard<std::mutex> lock(g_ranges_mutex);
        auto it = g_ranges.find(base);
        if (it == g_ranges.end()) return AVSG_EINVAL;
        r = it->second;
        g_ranges.erase(it);
    }
    const cudaError_t e = cudaHostUnregister(base);
    if (e != cudaSuccess) (void)cudaGetLastError();
    munmap(r.map_base, r.map_bytes);
    return e == cudaSuccess ? AVSG_OK : AVSG_ECUDA;
}

}  // extern "C"
