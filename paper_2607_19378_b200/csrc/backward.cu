// Helpers of the backward pass of the gated long convolution.  The gradients are themselves long convolutions
// (with the kernel read at the opposite displacement, or with the roles of signal and kernel exchanged), so the
// transform kernels are the forward's; what is new is bookkeeping: re-indexing kernels, zero-padding onto the
// transform grid, reading taps back from it, products and casts.  All of it is fp32 and pointwise.
#include "common.cuh"
#include "backward.cuh"

namespace hn {

constexpr int kBwdThreads = 256;

static int bwd_grid(long long items)
{
    static int sms = 0;
    if (!sms) {
        int dev = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (sms <= 0) sms = 148;
    }
    const long long want = (items + kBwdThreads - 1) / kBwdThreads, cap = (long long)sms * 16;
    return (int)(want < cap ? want : cap);
}

__device__ __forceinline__ int remap_index(int mode, int i, int G, int Ls, int shift)
{
    switch (mode) {
    case REMAP_PAD: return i;
    case REMAP_NEG: return i == 0 ? 0 : G - i;
    case REMAP_REV: return Ls - 1 - i;
    default: {
        int j = (i - shift) % Ls;
        return j < 0 ? j + Ls : j;
    }
    }
}

__global__ void __launch_bounds__(kBwdThreads) remap_kernel(RemapArgs r)
{
    const long long gvol = (long long)r.G[0] * r.G[1] * r.G[2], svol = (long long)r.Ls[0] * r.Ls[1] * r.Ls[2];
    const long long total = r.slices * gvol;
    for (long long e = (long long)blockIdx.x * kBwdThreads + threadIdx.x; e < total; e += (long long)gridDim.x * kBwdThreads) {
        const long long s = e / gvol, w = e % gvol;
        const int i2 = (int)(w % r.G[2]), i1 = (int)((w / r.G[2]) % r.G[1]), i0 = (int)(w / ((long long)r.G[2] * r.G[1]));
        const int j0 = remap_index(r.mode[0], i0, r.G[0], r.Ls[0], r.shift[0]);
        const int j1 = remap_index(r.mode[1], i1, r.G[1], r.Ls[1], r.shift[1]);
        const int j2 = remap_index(r.mode[2], i2, r.G[2], r.Ls[2], r.shift[2]);
        float val = 0.f;
        if (j0 >= 0 && j0 < r.Ls[0] && j1 >= 0 && j1 < r.Ls[1] && j2 >= 0 && j2 < r.Ls[2]) {
            const long long src = s * svol + ((long long)j0 * r.Ls[1] + j1) * r.Ls[2] + j2;
            if (r.a_bf16) {
                const bf16 *ab = reinterpret_cast<const bf16 *>(r.a);
                HN_G(ab + src, 2);
                val = __bfloat162float(ab[src]);
            } else {
                HN_G(r.a + src, 4);
                val = __ldg(r.a + src);
            }
            if (r.b) { HN_G(r.b + src, 4); val *= __ldg(r.b + src); }
        }
        if (r.out_bf16) {
            bf16 *ob = reinterpret_cast<bf16 *>(r.out);
            HN_G(ob + e, 2);
            ob[e] = __float2bfloat16_rn(val);
        } else {
            HN_G(r.out + e, 4);
            r.out[e] = val;
        }
    }
}

__global__ void fill_kernel(float *dst, float value, long long n)
{
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) { HN_G(dst + i, 4); dst[i] = value; }
}

template <typename T> __global__ void mul_cast_kernel(const float *a, const float *b, long long n, T *dst)
{
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x)
        { HN_G(a + i, 4); if (b) HN_G(b + i, 4); IO<T>::st(dst, i, b ? a[i] * b[i] : a[i]); }
}

__global__ void batch_sum_kernel(const float *src, long long nb, long long C, long long kvol, int set, float *acc)
{
    const long long total = C * kvol;
    for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (long long)gridDim.x * blockDim.x) {
        HN_G(acc + e, 4);
        float s = set ? 0.f : acc[e];
        for (long long b = 0; b < nb; ++b) { HN_G(src + b * total + e, 4); s += src[b * total + e]; }      // fixed order: the result does not depend on scheduling
        acc[e] = s;
    }
}

int launch_remap(const RemapArgs &r, cudaStream_t st)
{
    const long long total = r.slices * r.G[0] * r.G[1] * r.G[2];
    const int grid = bwd_grid(total);
    if (grid <= 0) return 0;
    remap_kernel<<<grid, kBwdThreads, 0, st>>>(r);
    return 1;
}

int launch_fill(float *dst, float value, long long n, cudaStream_t st)
{
    const int grid = bwd_grid(n);
    if (grid <= 0) return 0;
    fill_kernel<<<grid, kBwdThreads, 0, st>>>(dst, value, n);
    return 1;
}

int launch_mul_cast(const float *a, const float *b, long long n, int dtype, void *dst, cudaStream_t st)
{
    const int grid = bwd_grid(n);
    if (grid <= 0) return 0;
    if (dtype == 0) mul_cast_kernel<float><<<grid, kBwdThreads, 0, st>>>(a, b, n, (float *)dst);
    else mul_cast_kernel<bf16><<<grid, kBwdThreads, 0, st>>>(a, b, n, (bf16 *)dst);
    return 1;
}

int launch_batch_sum(const float *src, long long nb, long long C, long long kvol, bool set, float *acc, cudaStream_t st)
{
    const int grid = bwd_grid(C * kvol);
    if (grid <= 0) return 0;
    batch_sum_kernel<<<grid, kBwdThreads, 0, st>>>(src, nb, C, kvol, set ? 1 : 0, acc);
    return 1;
}

}  // namespace hn
