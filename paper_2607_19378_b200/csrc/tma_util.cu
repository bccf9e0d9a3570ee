// Tensor-map encoding for the kernels that use TMA (host side of tma_util.cuh).
#include <cstring>
#include "tma_util.cuh"

namespace hn {

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult qr;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qr) == cudaSuccess &&
            qr == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
        else
            cudaGetLastError();
    }
    return fn;
}

bool tma_available() { return encode_fn() != nullptr; }

bool tma_encode_3d(CUtensorMap *map, const void *base, bool bf16, const unsigned long long dims[3],
                   const unsigned long long strides[2], const unsigned box[3], int swizzle_bytes)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    if ((strides[0] % 16) || (strides[1] % 16) || ((uintptr_t)base % 16)) return false;
    if (swizzle_bytes != 0 && swizzle_bytes != 64 && swizzle_bytes != 128) return false;
    const cuuint64_t d[3] = {dims[0], dims[1], dims[2]};
    const cuuint64_t s[2] = {strides[0], strides[1]};
    const cuuint32_t b[3] = {box[0], box[1], box[2]};
    const cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<void *>(base), d, s, b,
              estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              swizzle_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : swizzle_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_NONE,
              CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool tma_encode_3d_cached(CUtensorMap *map, const void *base, bool bf16, const unsigned long long dims[3],
                          const unsigned long long strides[2], const unsigned box[3], int swizzle_bytes)
{
    struct Key {
        const void *base;
        unsigned long long dims[3], strides[2];
        unsigned box[3];
        int swizzle, bf16;
    };
    struct Entry { Key key; CUtensorMap map; bool used; };
    constexpr int kEntries = 16;
    static thread_local Entry cache[kEntries];
    Key k;
    memset(&k, 0, sizeof(k));
    k.base = base; k.swizzle = swizzle_bytes; k.bf16 = bf16 ? 1 : 0;
    for (int i = 0; i < 3; ++i) { k.dims[i] = dims[i]; k.box[i] = box[i]; }
    k.strides[0] = strides[0]; k.strides[1] = strides[1];
    unsigned long long h = (unsigned long long)(uintptr_t)base * 0x9E3779B97F4A7C15ull ^ dims[0] * 31 ^ dims[1] * 131 ^ dims[2] * 1031 ^
                           (unsigned long long)box[0] * 7 ^ (unsigned long long)box[1] * 13 ^ (unsigned long long)swizzle_bytes;
    Entry &e = cache[(h >> 7) % kEntries];
    if (e.used && memcmp(&e.key, &k, sizeof(k)) == 0) { *map = e.map; return true; }
    if (!tma_encode_3d(map, base, bf16, dims, strides, box, swizzle_bytes)) return false;
    e.key = k; e.map = *map; e.used = true;
    return true;
}

__global__ void bounded_wait_selftest_kernel(int polls, int *status)
{
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        fence_mbar_init();
    }
    __syncthreads();
    // nobody arrives on `bar`: the wait must run out and report it
    if (!mbar_wait(&bar, 0, polls)) {
        if (threadIdx.x == 0) atomicExch(status, 9);
    }
}

int tma_selftest_bounded_wait(int polls)
{
    int *d = nullptr, v = -1;
    if (polls < 1) polls = 1;
    if (polls > (1 << 16)) polls = 1 << 16;
    if (cudaMalloc(&d, sizeof(int)) != cudaSuccess) { cudaGetLastError(); return -1; }
    bool ok = cudaMemset(d, 0, sizeof(int)) == cudaSuccess;
    if (ok) {
        bounded_wait_selftest_kernel<<<1, 64>>>(polls, d);
        ok = cudaGetLastError() == cudaSuccess && cudaMemcpy(&v, d, sizeof(int), cudaMemcpyDeviceToHost) == cudaSuccess;
    }
    cudaFree(d);
    return ok ? v : -1;
}

}  // namespace hn
