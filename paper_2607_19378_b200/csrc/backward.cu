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

constexpr int kRemapPiece = 4096;
constexpr int kRemapRows = 8;

// A CTA takes kRemapRows consecutive output rows (slice, i0, i1) at a time: their source rows are worked out once per
// CTA and the threads walk the contiguous axis with one load per row in flight.  (One element per thread with a
// division and a modulo per element, and later one short row per CTA, kept so few bytes in flight that re-indexing
// the taps of volume3d took 7 ms: 0.6 TB/s.)  Long rows (1-D grids) are cut into pieces of kRemapPiece elements, one
// per blockIdx.y.
__global__ void __launch_bounds__(kBwdThreads) remap_kernel(RemapArgs r)
{
    const long long rows = r.slices * r.G[0] * r.G[1];
    const long long svol = (long long)r.Ls[0] * r.Ls[1] * r.Ls[2];
    const long long plane = (long long)r.G[0] * r.G[1];
    const int i2_0 = (int)blockIdx.y * kRemapPiece + threadIdx.x;
    const int i2_end = min(r.G[2], ((int)blockIdx.y + 1) * kRemapPiece);
    for (long long rb = (long long)blockIdx.x * kRemapRows; rb < rows; rb += (long long)gridDim.x * kRemapRows) {
        long long s = rb / plane;
        int w = (int)(rb - s * plane);
        int i0 = w / r.G[1], i1 = w - i0 * r.G[1];
        long long sbase[kRemapRows];
        bool row_in[kRemapRows];
#pragma unroll
        for (int k = 0; k < kRemapRows; ++k) {
            const int j0 = remap_index(r.mode[0], i0, r.G[0], r.Ls[0], r.shift[0]);
            const int j1 = remap_index(r.mode[1], i1, r.G[1], r.Ls[1], r.shift[1]);
            row_in[k] = rb + k < rows && j0 >= 0 && j0 < r.Ls[0] && j1 >= 0 && j1 < r.Ls[1];
            sbase[k] = s * svol + ((long long)j0 * r.Ls[1] + j1) * r.Ls[2];
            if (++i1 == r.G[1]) { i1 = 0; if (++i0 == r.G[0]) { i0 = 0; ++s; } }
        }
        for (int i2 = i2_0; i2 < i2_end; i2 += kBwdThreads) {
            const int j2 = remap_index(r.mode[2], i2, r.G[2], r.Ls[2], r.shift[2]);
            const bool col_in = j2 >= 0 && j2 < r.Ls[2];
            float val[kRemapRows];
#pragma unroll
            for (int k = 0; k < kRemapRows; ++k) {
                val[k] = 0.f;
                if (row_in[k] && col_in) {
                    const long long src = sbase[k] + j2;
                    if (r.a_bf16) {
                        const bf16 *ab = reinterpret_cast<const bf16 *>(r.a);
                        HN_G(ab + src, 2);
                        val[k] = __bfloat162float(ab[src]);
                    } else {
                        HN_G(r.a + src, 4);
                        val[k] = __ldg(r.a + src);
                    }
                }
            }
            if (r.b) {
#pragma unroll
                for (int k = 0; k < kRemapRows; ++k)
                    if (row_in[k] && col_in) {
                        const long long src = sbase[k] + j2;
                        if (r.a_bf16) {
                            const bf16 *bb = reinterpret_cast<const bf16 *>(r.b);
                            HN_G(bb + src, 2);
                            val[k] *= __bfloat162float(bb[src]);
                        } else {
                            HN_G(r.b + src, 4);
                            val[k] *= __ldg(r.b + src);
                        }
                    }
            }
#pragma unroll
            for (int k = 0; k < kRemapRows; ++k) {
                if (rb + k >= rows) break;
                const long long e = (rb + k) * r.G[2] + i2;
                if (r.out_bf16) {
                    bf16 *ob = reinterpret_cast<bf16 *>(r.out);
                    HN_G(ob + e, 2);
                    ob[e] = __float2bfloat16_rn(val[k]);
                } else {
                    HN_G(r.out + e, 4);
                    r.out[e] = val[k];
                }
            }
        }
    }
}

// Reversal along every axis with equal source and output extents is the reversal of the flattened slice:
// out[s][e] = a[s][N-1-e] (* b[s][N-1-e]).  One thread moves kRevUnroll elements, kBwdThreads apart, all loads issued
// before the first store: with 2- or 4-byte elements it takes that many loads in flight per thread to keep HBM busy
// (the general kernel above reaches 0.6 TB/s on the 2.1 GB of volume3d's taps, this one the copy rate).
constexpr int kRevUnroll = 16;

template <typename TA, typename TO>
__global__ void __launch_bounds__(kBwdThreads) reverse_kernel(const TA *a, const TA *b, TO *out, long long n)
{
    const long long base = (long long)blockIdx.y * n;
    const long long e0 = (long long)blockIdx.x * (kBwdThreads * kRevUnroll) + threadIdx.x;
    float val[kRevUnroll];
#pragma unroll
    for (int u = 0; u < kRevUnroll; ++u) {
        const long long e = e0 + (long long)u * kBwdThreads;
        val[u] = 0.f;
        if (e < n) { const long long src = base + n - 1 - e; HN_G(a + src, sizeof(TA)); val[u] = IO<TA>::ld(a, src); }
    }
    if (b) {
#pragma unroll
        for (int u = 0; u < kRevUnroll; ++u) {
            const long long e = e0 + (long long)u * kBwdThreads;
            if (e < n) { const long long src = base + n - 1 - e; HN_G(b + src, sizeof(TA)); val[u] *= IO<TA>::ld(b, src); }
        }
    }
#pragma unroll
    for (int u = 0; u < kRevUnroll; ++u) {
        const long long e = e0 + (long long)u * kBwdThreads;
        if (e < n) IO<TO>::st(out, base + e, val[u]);
    }
}

__global__ void fill_kernel(float *dst, float value, long long n)
{
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) { HN_G(dst + i, 4); dst[i] = value; }
}

template <typename T, typename TB> __global__ void mul_cast_kernel(const float *a, const TB *b, long long n, T *dst)
{
    // eight elements per thread and round, all loads before the first store
    constexpr int U = 8;
    const long long step = (long long)gridDim.x * blockDim.x * U;
    for (long long i0 = (long long)blockIdx.x * blockDim.x * U + threadIdx.x; i0 < n; i0 += step) {
        float v[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const long long i = i0 + (long long)u * blockDim.x;
            v[u] = 0.f;
            if (i < n) { HN_G(a + i, 4); v[u] = a[i]; }
        }
        if (b) {
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const long long i = i0 + (long long)u * blockDim.x;
                if (i < n) { HN_G(b + i, sizeof(TB)); v[u] *= IO<TB>::ld(b, i); }
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const long long i = i0 + (long long)u * blockDim.x;
            if (i < n) IO<T>::st(dst, i, v[u]);
        }
    }
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
    const long long rows = r.slices * r.G[0] * r.G[1];
    if (rows <= 0 || r.G[2] <= 0) return 0;
    bool flat_rev = r.slices <= 65535;
    for (int x = 0; x < 3; ++x)                            // an axis of one point maps 0 -> 0 in every mode but WRAP
        flat_rev = flat_rev && r.G[x] == r.Ls[x] && (r.mode[x] == REMAP_REV || (r.G[x] == 1 && r.mode[x] != REMAP_WRAP));
    if (flat_rev) {
        const long long n = (long long)r.G[0] * r.G[1] * r.G[2];
        const long long per = (long long)kBwdThreads * kRevUnroll;
        const dim3 grid((unsigned)((n + per - 1) / per), (unsigned)r.slices);
        if (r.a_bf16 && r.out_bf16) reverse_kernel<bf16, bf16><<<grid, kBwdThreads, 0, st>>>((const bf16 *)r.a, (const bf16 *)r.b, (bf16 *)r.out, n);
        else if (r.a_bf16) reverse_kernel<bf16, float><<<grid, kBwdThreads, 0, st>>>((const bf16 *)r.a, (const bf16 *)r.b, r.out, n);
        else if (r.out_bf16) reverse_kernel<float, bf16><<<grid, kBwdThreads, 0, st>>>(r.a, r.b, (bf16 *)r.out, n);
        else reverse_kernel<float, float><<<grid, kBwdThreads, 0, st>>>(r.a, r.b, r.out, n);
        return 1;
    }
    const long long cap = 1ll << 20;                       // CTAs; more rows than that are walked in a loop
    const unsigned pieces = (unsigned)((r.G[2] + kRemapPiece - 1) / kRemapPiece);      // <= 8192 for lines of up to 2^25 points
    const long long ctas = (rows + kRemapRows - 1) / kRemapRows;
    remap_kernel<<<dim3((unsigned)(ctas < cap ? ctas : cap), pieces), kBwdThreads, 0, st>>>(r);
    return 1;
}

int launch_fill(float *dst, float value, long long n, cudaStream_t st)
{
    const int grid = bwd_grid(n);
    if (grid <= 0) return 0;
    fill_kernel<<<grid, kBwdThreads, 0, st>>>(dst, value, n);
    return 1;
}

int launch_mul_cast(const float *a, const void *b, int b_dtype, long long n, int dtype, void *dst, cudaStream_t st)
{
    const int grid = bwd_grid((n + 7) / 8);
    if (grid <= 0) return 0;
    const bool bh = b && b_dtype != 0;
    if (dtype == 0 && !bh) mul_cast_kernel<float, float><<<grid, kBwdThreads, 0, st>>>(a, (const float *)b, n, (float *)dst);
    else if (dtype == 0) mul_cast_kernel<float, bf16><<<grid, kBwdThreads, 0, st>>>(a, (const bf16 *)b, n, (float *)dst);
    else if (!bh) mul_cast_kernel<bf16, float><<<grid, kBwdThreads, 0, st>>>(a, (const float *)b, n, (bf16 *)dst);
    else mul_cast_kernel<bf16, bf16><<<grid, kBwdThreads, 0, st>>>(a, (const bf16 *)b, n, (bf16 *)dst);
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
