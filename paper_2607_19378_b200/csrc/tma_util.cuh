// TMA helpers shared by the kernels that move tiles as tensor copies: mbarrier and
// cp.async.bulk.tensor wrappers (device) and tensor-map encoding (host).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <cstdint>

namespace hn {

// A wait on a barrier gives up after kWaitLimitNs of device time (read from the global nanosecond timer every
// 256 polls) or after kWaitLimit polls, whichever comes first.  A tile copy completes in microseconds.
constexpr int kWaitLimit = 1 << 22;
constexpr unsigned long long kWaitLimitNs = 1000000000ull;      // one second

__device__ __forceinline__ unsigned smem_u32(const void *p) { return (unsigned)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t *b, unsigned count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(smem_u32(b)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *b, unsigned bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(smem_u32(b)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *b, unsigned parity)
{
    unsigned ok;
    asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
                 : "=r"(ok) : "r"(smem_u32(b)), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long globaltimer_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;\n" : "=l"(t));
    return t;
}
// bounded wait; false if the phase did not complete within `limit` polls or kWaitLimitNs nanoseconds
__device__ __forceinline__ bool mbar_wait(uint64_t *b, unsigned parity, int limit = kWaitLimit)
{
    if (mbar_try_wait(b, parity)) return true;
    const unsigned long long t0 = globaltimer_ns();
    for (int i = 1; i < limit; ++i) {
        if (mbar_try_wait(b, parity)) return true;
        if ((i & 255) == 0 && globaltimer_ns() - t0 > kWaitLimitNs) return false;
    }
    return false;
}
__device__ __forceinline__ void tma_load_3d(void *dst, const CUtensorMap *map, uint64_t *bar, int x, int y, int z)
{
    asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];\n"
                 ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(x), "r"(y), "r"(z) : "memory");
}
__device__ __forceinline__ void tma_store_3d(const CUtensorMap *map, const void *src, int x, int y, int z)
{
    asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];\n"
                 ::"l"(map), "r"(smem_u32(src)), "r"(x), "r"(y), "r"(z) : "memory");
}
__device__ __forceinline__ void tma_commit() { asm volatile("cp.async.bulk.commit_group;\n" ::: "memory"); }
__device__ __forceinline__ void tma_wait_read0() { asm volatile("cp.async.bulk.wait_group.read 0;\n" ::: "memory"); }
__device__ __forceinline__ void tma_wait_all0() { asm volatile("cp.async.bulk.wait_group 0;\n" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory"); }
__device__ __forceinline__ void fence_mbar_init() { asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory"); }


// ---- host -----------------------------------------------------------------------------------------------------
// true if the driver offers tensor-map encoding (looked up once through the runtime)
bool tma_available();
// Self-test of the bounded wait: one CTA waits, for at most `polls` polls, on a barrier that nothing ever
// completes, and must come back with code 9 in the returned status word (0 would mean the wait "succeeded",
// -1 a CUDA error).  Blocking; allocates and frees one device word.
int tma_selftest_bounded_wait(int polls);
// Encodes a 3-D tiled map of fp32 (bf16 = false) or bf16 elements: dims and box in elements (innermost first),
// strides in bytes for dimensions 1 and 2, swizzle = bytes of one box row (64 or 128) or 0 for none.  False if the arguments
// break an alignment rule or the driver refuses.
bool tma_encode_3d(CUtensorMap *map, const void *base, bool bf16, const unsigned long long dims[3],
                   const unsigned long long strides[2], const unsigned box[3], int swizzle_bytes);
// The same through a small per-thread cache keyed by every argument: callers that pass the same tensors call after
// call (a training loop's fixed buffers) skip the driver's encoding.  Encoding reads no device memory, so a cached map
// stays valid as long as the key matches.
bool tma_encode_3d_cached(CUtensorMap *map, const void *base, bool bf16, const unsigned long long dims[3],
                          const unsigned long long strides[2], const unsigned box[3], int swizzle_bytes);

}  // namespace hn
