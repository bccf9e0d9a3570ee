// Pointwise stages of the full HyenaND operator, Eq. 2 of the paper (Section 3.2):
//
//     y = RMSNorm( Sigmoid(v) * ( K conv RMSNorm( l2(q) * SiLU(k) ) ) )
//
// Both normalisations and the l2 norm act per token across the C channels.  In the [B][C][L] layout a token's
// channels are L elements apart, so a thread owns one token and walks the channels: neighbouring threads read
// neighbouring tokens (coalesced), the per-token sums stay in registers, and the second walk over the channels
// (which writes the results) re-reads a tile that the first walk just brought into the caches.
// All arithmetic is fp32; the results that feed the long convolution stay fp32 (nothing is rounded to bf16 before
// the transforms); the one rounding to the I/O type happens at the final store of y.
#include "common.cuh"
#include "mixer.cuh"

namespace hn {

constexpr int kMixThreads = 256;
constexpr float kL2Floor = 1e-12f;

__device__ __forceinline__ float sigmoidf_(float x) { return 1.f / (1.f + __expf(-x)); }

template <typename T>
__global__ void __launch_bounds__(kMixThreads) mixer_pre_kernel(const T *q, const T *k, const T *v, const float *g_in,
                                                                float eps, long long nb, int C, long long L,
                                                                float *qz, float *kz, float *vz)
{
    const long long tokens = nb * L;
    for (long long t = (long long)blockIdx.x * kMixThreads + threadIdx.x; t < tokens; t += (long long)gridDim.x * kMixThreads) {
        const long long b = t / L, i = t % L;
        const long long base = b * C * L + i;
        float s1 = 0.f, s2 = 0.f;                       // sum q^2, sum (q SiLU(k))^2
        for (int c = 0; c < C; ++c) {
            const float qc = IO<T>::ld(q, base + c * L), kc = IO<T>::ld(k, base + c * L);
            const float sk = kc * sigmoidf_(kc);
            s1 = fmaf(qc, qc, s1);
            s2 = fmaf(qc * sk, qc * sk, s2);
        }
        const float inv_norm = 1.f / fmaxf(sqrtf(s1), kL2Floor);
        // mean_c (l2(q) SiLU(k))^2 = s2 / (C ||q||^2)
        const float scale = inv_norm * rsqrtf(s2 * inv_norm * inv_norm / (float)C + eps);
        for (int c = 0; c < C; ++c) {
            const float qc = IO<T>::ld(q, base + c * L), kc = IO<T>::ld(k, base + c * L), vc = IO<T>::ld(v, base + c * L);
            HN_G(g_in + c, 4); HN_G(kz + base + c * L, 4); HN_G(vz + base + c * L, 4); HN_G(qz + base + c * L, 4);
            kz[base + c * L] = qc * scale * __ldg(g_in + c);
            vz[base + c * L] = kc * sigmoidf_(kc);
            qz[base + c * L] = sigmoidf_(vc);
        }
    }
}

template <typename T>
__global__ void __launch_bounds__(kMixThreads) mixer_post_kernel(const float *o, const float *g_out, float eps, long long nb,
                                                                 int C, long long L, T *y)
{
    const long long tokens = nb * L;
    for (long long t = (long long)blockIdx.x * kMixThreads + threadIdx.x; t < tokens; t += (long long)gridDim.x * kMixThreads) {
        const long long b = t / L, i = t % L;
        const long long base = b * C * L + i;
        float s = 0.f;
        for (int c = 0; c < C; ++c) {
            HN_G(o + base + c * L, 4);
            const float oc = __ldg(o + base + c * L);
            s = fmaf(oc, oc, s);
        }
        const float scale = rsqrtf(s / (float)C + eps);
        for (int c = 0; c < C; ++c) { HN_G(g_out + c, 4); IO<T>::st(y, base + c * L, __ldg(o + base + c * L) * scale * __ldg(g_out + c)); }
    }
}

template <typename T> __global__ void widen_kernel(const T *src, long long n, float *dst)
{
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x)
        { HN_G(dst + i, 4); dst[i] = IO<T>::ld(src, i); }
}

static int mix_grid(long long items)
{
    static int sms = 0;
    if (!sms) {
        int dev = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (sms <= 0) sms = 148;
    }
    const long long want = (items + kMixThreads - 1) / kMixThreads, cap = (long long)sms * 8;
    return (int)(want < cap ? want : cap);
}

int launch_mixer_pre(const void *q, const void *k, const void *v, const float *g_in, float eps, int dtype,
                     long long nb, int C, long long L, float *qz, float *kz, float *vz, cudaStream_t st)
{
    const int grid = mix_grid(nb * L);
    if (grid <= 0) return 0;
    if (dtype == 0)
        mixer_pre_kernel<float><<<grid, kMixThreads, 0, st>>>((const float *)q, (const float *)k, (const float *)v, g_in, eps, nb, C, L, qz, kz, vz);
    else
        mixer_pre_kernel<bf16><<<grid, kMixThreads, 0, st>>>((const bf16 *)q, (const bf16 *)k, (const bf16 *)v, g_in, eps, nb, C, L, qz, kz, vz);
    return 1;
}

int launch_mixer_post(const float *o, const float *g_out, float eps, int dtype, long long nb, int C, long long L,
                      void *y, cudaStream_t st)
{
    const int grid = mix_grid(nb * L);
    if (grid <= 0) return 0;
    if (dtype == 0) mixer_post_kernel<float><<<grid, kMixThreads, 0, st>>>(o, g_out, eps, nb, C, L, (float *)y);
    else mixer_post_kernel<bf16><<<grid, kMixThreads, 0, st>>>(o, g_out, eps, nb, C, L, (bf16 *)y);
    return 1;
}

int launch_widen(const void *src, int dtype, long long n, float *dst, cudaStream_t st)
{
    const int grid = mix_grid(n);
    if (grid <= 0) return 0;
    if (dtype == 0) widen_kernel<float><<<grid, kMixThreads, 0, st>>>((const float *)src, n, dst);
    else widen_kernel<bf16><<<grid, kMixThreads, 0, st>>>((const bf16 *)src, n, dst);
    return 1;
}

}  // namespace hn
