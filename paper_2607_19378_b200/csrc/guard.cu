// Guarded device allocations and the environment switches of a plan (host code only).
#include <stdlib.h>
#include <string.h>

#include <vector>

#include <nvtx3/nvToolsExt.h>

#include "common.cuh"

namespace hn {

static const unsigned char kGuardByte = 0xA5;

Switches read_switches()
{
    Switches s;
    s.force_generic = getenv("HYENAND_FORCE_GENERIC") != nullptr;
    s.generic_rows = getenv("HYENAND_GENERIC_ROWS") != nullptr;
    s.generic_core = getenv("HYENAND_GENERIC_CORE") != nullptr;
    s.no_tma = getenv("HYENAND_NO_TMA") != nullptr;
    s.nvtx = getenv("HYENAND_NVTX") != nullptr;
    return s;
}

// ---- checked build: hooks of the translation units ----------------------------------------------------------
static DbgHook g_dbg_hooks[32];
static const char *g_dbg_files[32];
static int g_dbg_n = 0;

void dbg_register(DbgHook hook, const char *file)
{
    if (g_dbg_n < 32) { g_dbg_hooks[g_dbg_n] = hook; g_dbg_files[g_dbg_n] = file; ++g_dbg_n; }
}

static DbgRanges g_dbg_last;

void dbg_set_ranges(const DbgRanges &r)
{
    g_dbg_last = r;
    for (int i = 0; i < g_dbg_n; ++i) g_dbg_hooks[i](&r, nullptr);
}

void dbg_append_range(const void *ptr, size_t bytes)
{
    if (!ptr || !bytes || g_dbg_last.n >= kDbgRanges) return;
    g_dbg_last.lo[g_dbg_last.n] = (unsigned long long)ptr;
    g_dbg_last.hi[g_dbg_last.n] = (unsigned long long)ptr + bytes;
    ++g_dbg_last.n;
    dbg_set_ranges(g_dbg_last);
}

DbgReport dbg_collect()
{
    DbgReport rep{0, 0, 0, nullptr};
    for (int i = 0; i < g_dbg_n; ++i) {
        unsigned long long c[4] = {0, 0, 0, 0};
        g_dbg_hooks[i](nullptr, c);
        if (c[0] && !rep.count) { rep.first_address = c[1]; rep.first_line = (int)c[2]; rep.file = g_dbg_files[i]; }
        rep.count += c[0];
    }
    return rep;
}

void nvtx_push(const char *name) { nvtxRangePushA(name); }
void nvtx_pop() { nvtxRangePop(); }

cudaError_t guarded_alloc(GuardedAllocs *g, void **ptr, size_t bytes)
{
    *ptr = nullptr;
    if (g->n >= kMaxGuarded) return cudaErrorMemoryAllocation;
    if (bytes == 0) bytes = 16;
    const size_t body = (bytes + 255) & ~(size_t)255;          // the upper band starts on a 256-byte boundary too
    unsigned char *base = nullptr;
    cudaError_t e = cudaMalloc((void **)&base, body + 2 * kGuardBytes);
    if (e != cudaSuccess) return e;
    e = cudaMemset(base, kGuardByte, kGuardBytes);
    if (e == cudaSuccess) e = cudaMemset(base + kGuardBytes + bytes, kGuardByte, body - bytes + kGuardBytes);
    if (e != cudaSuccess) { cudaFree(base); return e; }
    g->recs[g->n].base = base;
    g->recs[g->n].bytes = bytes;
    ++g->n;
    *ptr = base + kGuardBytes;
    return cudaSuccess;
}

void guarded_free_all(GuardedAllocs *g)
{
    for (int i = 0; i < g->n; ++i) cudaFree(g->recs[i].base);
    g->n = 0;
}

long long guard_damage(const GuardedAllocs *g)
{
    std::vector<unsigned char> host(kGuardBytes + 256);
    long long bad = 0;
    for (int i = 0; i < g->n; ++i) {
        const GuardedAllocs::Rec &r = g->recs[i];
        const size_t body = (r.bytes + 255) & ~(size_t)255;
        const size_t upper = body - r.bytes + kGuardBytes;
        if (cudaMemcpy(host.data(), r.base, kGuardBytes, cudaMemcpyDeviceToHost) != cudaSuccess) return -1;
        for (size_t b = 0; b < kGuardBytes; ++b) bad += host[b] != kGuardByte;
        if (cudaMemcpy(host.data(), r.base + kGuardBytes + r.bytes, upper, cudaMemcpyDeviceToHost) != cudaSuccess) return -1;
        for (size_t b = 0; b < upper; ++b) bad += host[b] != kGuardByte;
    }
    return bad;
}

}  // namespace hn
