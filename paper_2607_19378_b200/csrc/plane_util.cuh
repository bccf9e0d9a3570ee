// Device helpers shared by the plane-fused 3-D kernels and the fused 2-D kernel.
#pragma once
#include "common.cuh"
#include "wfft.cuh"

namespace hn {

constexpr int kPlaneThreads = 512;

// lines start on 16-byte boundaries (asynchronous 16-byte copies land in them) and two
// neighbouring lines do not share banks: stride = 8 mod 16 complex numbers
__host__ __device__ constexpr int plane_ls(int n) { return ((phys_max(n) + 1 + 7) / 16) * 16 + 8; }

// Ask the memory system to bring [ptr, ptr + bytes) into L2, one prefetch per 128-byte line, the lines dealt out to
// the CTA's threads (a handful of plain prefetch instructions per thread; a bulk prefetch per thread is executed lane
// by lane and held the issuing warps up for thousands of cycles).  The CTA issues it for the plane it will work on
// next, so that plane's loads hit L2.
__device__ __forceinline__ void prefetch_l2(const void *ptr, long long bytes, int tid)
{
    const char *b = reinterpret_cast<const char *>(ptr);
    for (long long o = (long long)tid * 128; o < bytes; o += (long long)kPlaneThreads * 128) {
        HN_G(b + o, 1);
        asm volatile("prefetch.global.L2 [%0];\n" ::"l"(b + o) : "memory");
    }
}

__device__ __forceinline__ void cp_async16(void *smem_dst, const void *gmem_src)
{
    const unsigned d = (unsigned)__cvta_generic_to_shared(smem_dst);
    HN_G(gmem_src, 16);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(d), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;\n" ::: "memory"); }

// Copy n bytes starting at src (aligned to 2 or 4 bytes only: rows of odd length) into shared
// memory with 16-byte copies of the surrounding aligned chunks: byte k of the row lands at
// dst + (src & 15) + k.  [lo, hi) bounds the tensor; a chunk that would cross it (only at the
// two ends of the tensor) is filled 2 bytes at a time.  TPL lanes cooperate.
template <int TPL>
__device__ __forceinline__ void stage_row(unsigned char *dst, const unsigned char *src, int n,
                                          const unsigned char *lo, const unsigned char *hi, int l)
{
    const unsigned char *a = src - ((unsigned long long)src & 15ull);
    const int nch = (int)((src + n - a + 15) >> 4);
    if (a >= lo && a + 16 * nch <= hi) {                   // all but the first and last rows of a tensor
        for (int c = l; c < nch; c += TPL) cp_async16(dst + 16 * c, a + 16 * c);
        return;
    }
    for (int c = l; c < nch; c += TPL) {
        const unsigned char *g = a + 16 * c;
        if (g >= lo && g + 16 <= hi) cp_async16(dst + 16 * c, g);
        else {
            for (int b = 0; b < 16; b += 2)
                if (g + b >= src && g + b < src + n) {
                    HN_G(g + b, 2);
                    *reinterpret_cast<unsigned short *>(dst + 16 * c + b) = *reinterpret_cast<const unsigned short *>(g + b);
                }
        }
    }
}
// The same copy for rows of at most MAXB bytes: the chunk loop has a compile-time trip count, so every copy is one
// predicated instruction with constant offsets.
template <int TPL, int MAXB>
__device__ __forceinline__ void stage_row_u(unsigned char *dst, const unsigned char *src, int n,
                                            const unsigned char *lo, const unsigned char *hi, int l)
{
    const unsigned char *a = src - ((unsigned long long)src & 15ull);
    const int nch = (int)((src + n - a + 15) >> 4);
    if (a >= lo && a + 16 * nch <= hi) {
        constexpr int MAXCH = (MAXB + 15) / 16 + 1;
        unsigned char *d = dst + 16 * l;
        const unsigned char *g = a + 16 * l;
        const int left = nch - l;
#pragma unroll
        for (int t = 0; t < (MAXCH + TPL - 1) / TPL; ++t)
            if (t * TPL < left) cp_async16(d + 16 * TPL * t, g + 16 * TPL * t);
        return;
    }
    stage_row<TPL>(dst, src, n, lo, hi, l);
}
template <typename T> __device__ __forceinline__ float staged(const unsigned char *row, int off, int i)
{
    if constexpr (sizeof(T) == 4) return *reinterpret_cast<const float *>(row + off + 4 * i);
    else return __bfloat162float(*reinterpret_cast<const bf16 *>(row + off + 2 * i));
}

// Zero elements [from, to) of a staged row (element i sits at row + off + i*sizeof(T)); used to blank
// the padding positions once so that the transform's input functor needs no bounds test.
template <typename T, int TPL>
__device__ __forceinline__ void zero_staged(unsigned char *row, int off, int from, int to, int l)
{
    for (int i = from + l; i < to; i += TPL) *reinterpret_cast<T *>(row + off + (int)sizeof(T) * i) = T(0.f);
}

// Engines with 8 lanes per line put two lines into each half warp.  When both lines walk a column
// store (consecutive columns per lane, one row or column offset per line), the two must sit D
// entries apart to use different banks: spread_pair<D>(g) renumbers the groups so that g and g ^ 1
// get numbers D apart (a bijection on every aligned block of 2*D groups).
template <int D> __host__ __device__ __forceinline__ constexpr int spread_pair(int g)
{
    return ((g >> 1) & (D - 1)) | ((g & 1) * D) | (g & ~(2 * D - 1));
}

// 16 bytes of gate values or results: VEC elements of T
template <typename T> struct Vec16;
template <> struct Vec16<float> {
    static constexpr int VEC = 4;
    static __device__ __forceinline__ void unpack(const uint4 &u, float (&f)[4])
    {
        f[0] = __uint_as_float(u.x); f[1] = __uint_as_float(u.y); f[2] = __uint_as_float(u.z); f[3] = __uint_as_float(u.w);
    }
    static __device__ __forceinline__ uint4 pack(const float (&f)[4])
    {
        return make_uint4(__float_as_uint(f[0]), __float_as_uint(f[1]), __float_as_uint(f[2]), __float_as_uint(f[3]));
    }
};
template <> struct Vec16<bf16> {
    static constexpr int VEC = 8;
    static __device__ __forceinline__ void unpack(const uint4 &u, float (&f)[8])
    {
        const unsigned w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) { f[2 * i] = __uint_as_float(w[i] << 16); f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u); }
    }
    static __device__ __forceinline__ uint4 pack(const float (&f)[8])
    {
        unsigned w[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const __nv_bfloat162 h = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
            w[i] = *reinterpret_cast<const unsigned *>(&h);
        }
        return make_uint4(w[0], w[1], w[2], w[3]);
    }
};

// Twiddle source of the P-point transforms of a plane kernel: registers when the plan has two
// equal passes (the twiddles of the second pass then depend on the lane only), else per-pass
// tables in shared memory.
template <int LOG2P, bool INV> struct PlaneTw {
    using F = WF<LOG2P, INV>;
    static constexpr bool HOIST = F::NP == 2 && (WPlan<LOG2P>::R[0] == WPlan<LOG2P>::R[1] || (LOG2P == 7 && !INV));
    static constexpr int TABLE = HOIST ? 0 : PassTw<LOG2P, INV>::TOTAL;   // shared-memory entries needed
    typename F::template Hoist<F::NP - 1> hw;
    PassTw<LOG2P, INV> pt;
    // full: N-point table in shared memory (already filled); tab: room for TABLE entries
    __device__ __forceinline__ void init(int l, const float2 *full, float2 *tab, int tid, int nthr)
    {
        pt.base = tab;
        if constexpr (HOIST) hw.load(l, full);
        else {
            for (int s = 1; s < F::NP; ++s) {
                const int ns = F::ns(s), rad = F::radix(s), off = PassTw<LOG2P, INV>::offset(s);
                for (int e = tid; e < (rad - 1) * ns; e += nthr) {
                    const int r = e / ns + 1, k = e % ns;
                    tab[off + e] = full[r * k * ((1 << LOG2P) / (ns * rad))];
                }
            }
        }
    }
    template <int S> __device__ __forceinline__ float2 get(int i, int r, int k, int t) const
    {
        if constexpr (HOIST) return hw.template get<S>(i, r, k, t);
        else return pt.template get<S>(i, r, k, t);
    }
};

}  // namespace hn
