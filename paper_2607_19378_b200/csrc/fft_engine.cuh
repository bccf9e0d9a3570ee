// Shared-memory complex FFT engine (fp32) for power-of-two line lengths.
//
// A "line" is N complex points in shared memory.  Transforms are Stockham
// autosort passes of radix 4/8/16 (radix 2 only for N = 2): every pass reads
// R points at stride N/R, applies the pass twiddles, runs an R-point DFT in
// registers and writes R points back, so data leaves registers once per pass.
// Lines are stored with one pad element every 16 (phys()) so that both the
// contiguous reads and the strided writes of a pass are bank-conflict free.
//
// Pruning: the padded convolution (Section 3.2.1; Appendix B.1, Eq. 11-13 of
// the paper) transforms inputs whose upper half is zero and keeps only the
// lower half of every inverse.  PRUNE_IN drops the arithmetic on the zero half
// in the first pass, PRUNE_OUT skips the unused outputs of the last pass.
#pragma once
#include <type_traits>
#include <cuda_runtime.h>
#include "common.cuh"

namespace hn {

enum { PRUNE_NONE = 0, PRUNE_IN = 1, PRUNE_OUT = 2 };

__host__ __device__ __forceinline__ constexpr int phys(int i) { return i + (i >> 4); }
// shared-memory floats2 needed for one line of n points (odd, so lines do not alias banks)
// largest skewed position + 1 of an n-point line under any engine (the warp engine skews short
// lines by i >> 3)
__host__ __device__ __forceinline__ constexpr int phys_max(int n) { return n <= 128 ? n + (n >> 3) : n + (n >> 4); }
__host__ __device__ __forceinline__ constexpr int line_stride(int n) { return (phys_max(n) + 1) | 1; }

__device__ __forceinline__ float2 cadd(float2 a, float2 b) { return make_float2(a.x + b.x, a.y + b.y); }
__device__ __forceinline__ float2 csub(float2 a, float2 b) { return make_float2(a.x - b.x, a.y - b.y); }
__device__ __forceinline__ float2 cmul(float2 a, float2 w)
{
    return make_float2(fmaf(a.x, w.x, -a.y * w.y), fmaf(a.x, w.y, a.y * w.x));
}
__device__ __forceinline__ float2 cmulc(float2 a, float2 w)   // a * conj(w)
{
    return make_float2(fmaf(a.x, w.x, a.y * w.y), fmaf(a.y, w.x, -a.x * w.y));
}
// multiply by -i (forward transforms) or +i (inverse)
template <bool INV> __device__ __forceinline__ float2 rot90(float2 a)
{
    return INV ? make_float2(-a.y, a.x) : make_float2(a.y, -a.x);
}

#define HN_SQ2 0.70710678118654752440f
#define HN_C8  0.92387953251128675613f   // cos(pi/8)
#define HN_S8  0.38268343236508977173f   // sin(pi/8)

// a * W_16^T (forward sign; conjugate for INV), T compile-time
template <int T, bool INV> __device__ __forceinline__ float2 mul_w16(float2 a)
{
    constexpr int t = T & 15;
    if constexpr (t == 0) return a;
    else if constexpr (t == 4) return rot90<INV>(a);
    else if constexpr (t == 8) return make_float2(-a.x, -a.y);
    else if constexpr (t == 12) return rot90<!INV>(a);
    else if constexpr (t == 2) {
        return INV ? make_float2((a.x - a.y) * HN_SQ2, (a.x + a.y) * HN_SQ2)
                   : make_float2((a.x + a.y) * HN_SQ2, (a.y - a.x) * HN_SQ2);
    } else if constexpr (t == 6) {
        return INV ? make_float2(-(a.x + a.y) * HN_SQ2, (a.x - a.y) * HN_SQ2)
                   : make_float2((a.y - a.x) * HN_SQ2, -(a.x + a.y) * HN_SQ2);
    } else if constexpr (t == 10) {
        float2 m = mul_w16<2, INV>(a); return make_float2(-m.x, -m.y);
    } else if constexpr (t == 14) {
        float2 m = mul_w16<6, INV>(a); return make_float2(-m.x, -m.y);
    } else {
        // odd powers: cos/sin of t*pi/8
        constexpr float c = (t == 1 || t == 15) ? HN_C8 : (t == 3 || t == 13) ? HN_S8
                          : (t == 5 || t == 11) ? -HN_S8 : -HN_C8;
        constexpr float s0 = (t == 1 || t == 7) ? HN_S8 : (t == 3 || t == 5) ? HN_C8
                           : (t == 9 || t == 15) ? -HN_S8 : -HN_C8;     // sin(t*pi/8)
        constexpr float s = INV ? s0 : -s0;                              // forward: e^{-i..}
        return make_float2(fmaf(a.x, c, -a.y * s), fmaf(a.x, s, a.y * c));
    }
}

// W_16^T split as rho * c * (1 + i tau): rho a power of -i (free), c in {1, cos(pi/8), sqrt(1/2)} and
// tau in {0, +-tan(pi/8), +-1}.  w16_unscaled returns rho (1 + i tau) a (two fused multiply-adds at most); the factor
// c is left to the butterfly that consumes the value, where it turns an addition into a fused multiply-add.
#define HN_T8 0.41421356237309504880f   // tan(pi/8)
template <int T> __host__ __device__ constexpr float w16_scale()
{
    constexpr int t = T & 15;
    return (t % 4 == 0) ? 1.f : (t % 2 == 0 ? HN_SQ2 : HN_C8);
}
template <int T, bool INV> __device__ __forceinline__ float2 w16_unscaled(float2 a)
{
    constexpr int t = T & 15;
    // forward factor exp(-2 pi i t / 16): quarter turns q (rho = (-i)^q) and tau
    constexpr int qf = (t == 0 || t == 1 || t == 2 || t == 15) ? 0 : (t >= 3 && t <= 6) ? 1 : (t >= 7 && t <= 10) ? 2 : 3;
    constexpr float tf = (t % 4 == 0) ? 0.f : (t % 4 == 2) ? -1.f : (t % 4 == 1) ? -HN_T8 : HN_T8;
    constexpr int q = INV ? ((4 - qf) & 3) : qf;
    constexpr float tau = INV ? -tf : tf;
    float2 v = a;
    if constexpr (tau != 0.f) v = make_float2(fmaf(-tau, a.y, a.x), fmaf(tau, a.x, a.y));
    if constexpr (q == 0) return v;
    else if constexpr (q == 1) return make_float2(v.y, -v.x);
    else if constexpr (q == 2) return make_float2(-v.x, -v.y);
    else return make_float2(-v.y, v.x);
}

__device__ __forceinline__ float2 fma2(float s, float2 a, float2 b) { return make_float2(fmaf(s, a.x, b.x), fmaf(s, a.y, b.y)); }

// ---- register DFTs, natural order in and out ------------------------------------

template <bool INV, int PR> __device__ __forceinline__ void dft2(float2 &a, float2 &b)
{
    if constexpr (PR == PRUNE_IN) { b = a; }
    else if constexpr (PR == PRUNE_OUT) { a = cadd(a, b); }
    else { float2 t = a; a = cadd(t, b); b = csub(t, b); }
}

template <bool INV, int PR>
__device__ __forceinline__ void dft4(float2 &a0, float2 &a1, float2 &a2, float2 &a3)
{
    if constexpr (PR == PRUNE_IN) {            // a2 = a3 = 0
        float2 r = rot90<INV>(a1);
        float2 x0 = cadd(a0, a1), x2 = csub(a0, a1);
        float2 x1 = cadd(a0, r), x3 = csub(a0, r);
        a0 = x0; a1 = x1; a2 = x2; a3 = x3;
    } else {
        float2 t0 = cadd(a0, a2), t1 = csub(a0, a2);
        float2 t2 = cadd(a1, a3), t3 = rot90<INV>(csub(a1, a3));
        a0 = cadd(t0, t2);
        a1 = cadd(t1, t3);
        if constexpr (PR != PRUNE_OUT) { a2 = csub(t0, t2); a3 = csub(t1, t3); }
    }
}

// 4-point transform of a0, W^T1 a1, W^T2 a2, W^T3 a3 (W = W_16): the scale factors of the twiddles ride on the
// butterflies' fused multiply-adds.
template <bool INV, int PR, int T1, int T2, int T3>
__device__ __forceinline__ void dft4_tw(float2 &a0, float2 &a1, float2 &a2, float2 &a3)
{
    constexpr float s1 = w16_scale<T1>(), s2 = w16_scale<T2>(), s3 = w16_scale<T3>(), s31 = s3 / s1;
    const float2 m1 = w16_unscaled<T1, INV>(a1), m2 = w16_unscaled<T2, INV>(a2), m3 = w16_unscaled<T3, INV>(a3);
    const float2 t0 = make_float2(fmaf(s2, m2.x, a0.x), fmaf(s2, m2.y, a0.y));
    const float2 t1 = make_float2(fmaf(-s2, m2.x, a0.x), fmaf(-s2, m2.y, a0.y));
    const float2 u2 = make_float2(fmaf(s31, m3.x, m1.x), fmaf(s31, m3.y, m1.y));
    const float2 r3 = rot90<INV>(make_float2(fmaf(-s31, m3.x, m1.x), fmaf(-s31, m3.y, m1.y)));
    a0 = make_float2(fmaf(s1, u2.x, t0.x), fmaf(s1, u2.y, t0.y));
    a1 = make_float2(fmaf(s1, r3.x, t1.x), fmaf(s1, r3.y, t1.y));
    if constexpr (PR != PRUNE_OUT) {
        a2 = make_float2(fmaf(-s1, u2.x, t0.x), fmaf(-s1, u2.y, t0.y));
        a3 = make_float2(fmaf(-s1, r3.x, t1.x), fmaf(-s1, r3.y, t1.y));
    }
}

template <bool INV, int PR> __device__ __forceinline__ void dft8(float2 (&x)[8])
{
    // evens / odds as two 4-point transforms (inputs 4..7 are zero under PRUNE_IN)
    constexpr int P4 = (PR == PRUNE_IN) ? PRUNE_IN : PRUNE_NONE;
    float2 e0 = x[0], e1 = x[2], e2 = x[4], e3 = x[6];
    float2 o0 = x[1], o1 = x[3], o2 = x[5], o3 = x[7];
    dft4<INV, P4>(e0, e1, e2, e3);
    dft4<INV, P4>(o0, o1, o2, o3);
    // W8^1 and W8^3 without their factor sqrt(1/2), which rides on the last additions
    o1 = w16_unscaled<2, INV>(o1);
    o2 = mul_w16<4, INV>(o2);
    o3 = w16_unscaled<6, INV>(o3);
    x[0] = cadd(e0, o0); x[1] = fma2(HN_SQ2, o1, e1); x[2] = cadd(e2, o2); x[3] = fma2(HN_SQ2, o3, e3);
    if constexpr (PR != PRUNE_OUT) {
        x[4] = csub(e0, o0); x[5] = fma2(-HN_SQ2, o1, e1); x[6] = csub(e2, o2); x[7] = fma2(-HN_SQ2, o3, e3);
    }
}

template <bool INV, int PR> __device__ __forceinline__ void dft16(float2 (&x)[16])
{
    // n = 4*n1 + n2, k = k1 + 4*k2: 4-point transforms over n1, twiddle W16^(n2*k1),
    // 4-point transforms over n2.
    constexpr int PIN = (PR == PRUNE_IN) ? PRUNE_IN : PRUNE_NONE;
    constexpr int POUT = (PR == PRUNE_OUT) ? PRUNE_OUT : PRUNE_NONE;
    float2 a[4][4];                                  // a[n2][k1]
#pragma unroll
    for (int n2 = 0; n2 < 4; ++n2) {
        a[n2][0] = x[n2]; a[n2][1] = x[n2 + 4]; a[n2][2] = x[n2 + 8]; a[n2][3] = x[n2 + 12];
        dft4<INV, PIN>(a[n2][0], a[n2][1], a[n2][2], a[n2][3]);
    }
    // column k1 takes a[n2][k1] W16^(n2*k1), n2 = 1..3
    dft4<INV, POUT>(a[0][0], a[1][0], a[2][0], a[3][0]);
    dft4_tw<INV, POUT, 1, 2, 3>(a[0][1], a[1][1], a[2][1], a[3][1]);
    dft4_tw<INV, POUT, 2, 4, 6>(a[0][2], a[1][2], a[2][2], a[3][2]);
    dft4_tw<INV, POUT, 3, 6, 9>(a[0][3], a[1][3], a[2][3], a[3][3]);
#pragma unroll
    for (int k1 = 0; k1 < 4; ++k1) {
        x[k1] = a[0][k1]; x[k1 + 4] = a[1][k1];
        if constexpr (PR != PRUNE_OUT) { x[k1 + 8] = a[2][k1]; x[k1 + 12] = a[3][k1]; }
    }
}

// cos and sin of 2 pi t / 32
__host__ __device__ constexpr float w32_cos(int t)
{
    t &= 31;
    if (t > 16) t = 32 - t;
    const bool neg = t > 8;
    if (neg) t = 16 - t;
    const float v = t == 0 ? 1.f : t == 1 ? 0.98078528040323044913f : t == 2 ? 0.92387953251128675613f
                  : t == 3 ? 0.83146961230254523708f : t == 4 ? 0.70710678118654752440f
                  : t == 5 ? 0.55557023301960222474f : t == 6 ? 0.38268343236508977173f
                  : t == 7 ? 0.19509032201612826785f : 0.f;
    return neg ? -v : v;
}
__host__ __device__ constexpr float w32_sin(int t) { return w32_cos(t - 8); }

// a * W_32^T (forward sign; conjugate for INV), T compile-time
template <int T, bool INV> __device__ __forceinline__ float2 mul_w32(float2 a)
{
    constexpr int t = T & 31;
    if constexpr (t % 2 == 0) return mul_w16<t / 2, INV>(a);
    else {
        constexpr float c = w32_cos(t);
        constexpr float s = INV ? w32_sin(t) : -w32_sin(t);
        return make_float2(fmaf(a.x, c, -a.y * s), fmaf(a.x, s, a.y * c));
    }
}

// W_32^T split as rho * c * (1 + i tau) like the W_16 factors above: T = 8 q + r with r in (-4, 4], rho = (-i)^q,
// c = cos(r pi/16), tau = -tan(r pi/16) (forward sign; conjugate for INV).
template <int T> __host__ __device__ constexpr int w32_res() { return (((T & 31) + 3) & 7) - 3; }
template <int T> __host__ __device__ constexpr float w32_scale() { return w32_cos(w32_res<T>()); }
template <int T, bool INV> __device__ __forceinline__ float2 w32_unscaled(float2 a)
{
    constexpr int r = w32_res<T>();
    constexpr int qf = ((((T & 31) - r) / 8) & 3);
    constexpr float tf = r == 0 ? 0.f : r == 4 ? -1.f : -w32_sin(r) / w32_cos(r);
    constexpr int q = INV ? ((4 - qf) & 3) : qf;
    constexpr float tau = INV ? -tf : tf;
    float2 v = a;
    if constexpr (tau != 0.f) v = make_float2(fmaf(-tau, a.y, a.x), fmaf(tau, a.x, a.y));
    if constexpr (q == 0) return v;
    else if constexpr (q == 1) return make_float2(v.y, -v.x);
    else if constexpr (q == 2) return make_float2(-v.x, -v.y);
    else return make_float2(-v.y, v.x);
}

// 8-point transform of c[n] W_32^(n K1), n = 0..7: every scale factor (of the outer twiddles and of the two
// sqrt(1/2) twiddles inside) rides on a fused multiply-add of the butterflies.
template <bool INV, int PR, int K1> __device__ __forceinline__ void dft8_tw(float2 (&c)[8])
{
    constexpr float s1 = w32_scale<K1>(), s2 = w32_scale<2 * K1>(), s3 = w32_scale<3 * K1>(), s4 = w32_scale<4 * K1>(),
                    s5 = w32_scale<5 * K1>(), s6 = w32_scale<6 * K1>(), s7 = w32_scale<7 * K1>();
    const float2 m0 = c[0];
    const float2 m1 = w32_unscaled<K1, INV>(c[1]), m2 = w32_unscaled<2 * K1, INV>(c[2]), m3 = w32_unscaled<3 * K1, INV>(c[3]),
                 m4 = w32_unscaled<4 * K1, INV>(c[4]), m5 = w32_unscaled<5 * K1, INV>(c[5]), m6 = w32_unscaled<6 * K1, INV>(c[6]),
                 m7 = w32_unscaled<7 * K1, INV>(c[7]);
    // evens: true values
    const float2 t0 = fma2(s4, m4, m0), t1 = fma2(-s4, m4, m0);
    const float2 u2 = fma2(s6 / s2, m6, m2), r3 = rot90<INV>(fma2(-s6 / s2, m6, m2));
    const float2 e0 = fma2(s2, u2, t0), e1 = fma2(s2, r3, t1), e2 = fma2(-s2, u2, t0), e3 = fma2(-s2, r3, t1);
    // odds: values divided by s1
    const float2 v0 = fma2(s5 / s1, m5, m1), v1 = fma2(-s5 / s1, m5, m1);
    const float2 w2 = fma2(s7 / s3, m7, m3), w3 = rot90<INV>(fma2(-s7 / s3, m7, m3));
    const float2 o0 = fma2(s3 / s1, w2, v0), o1 = fma2(s3 / s1, w3, v1), o2 = fma2(-s3 / s1, w2, v0), o3 = fma2(-s3 / s1, w3, v1);
    const float2 p1 = w16_unscaled<2, INV>(o1), p2 = w16_unscaled<4, INV>(o2), p3 = w16_unscaled<6, INV>(o3);
    constexpr float sq = s1 * HN_SQ2;
    c[0] = fma2(s1, o0, e0); c[1] = fma2(sq, p1, e1); c[2] = fma2(s1, p2, e2); c[3] = fma2(sq, p3, e3);
    if constexpr (PR != PRUNE_OUT) {
        c[4] = fma2(-s1, o0, e0); c[5] = fma2(-sq, p1, e1); c[6] = fma2(-s1, p2, e2); c[7] = fma2(-sq, p3, e3);
    }
}

template <int N2, bool INV> __device__ __forceinline__ void tw32_row(float2 (&a)[4])
{
    a[1] = mul_w32<N2, INV>(a[1]); a[2] = mul_w32<2 * N2, INV>(a[2]); a[3] = mul_w32<3 * N2, INV>(a[3]);
}

template <bool INV, int PR> __device__ __forceinline__ void dft32(float2 (&x)[32])
{
    // n = 8*n1 + n2, k = k1 + 4*k2: 4-point transforms over n1, twiddle W32^(n2*k1),
    // 8-point transforms over n2.
    constexpr int PIN = (PR == PRUNE_IN) ? PRUNE_IN : PRUNE_NONE;
    constexpr int POUT = (PR == PRUNE_OUT) ? PRUNE_OUT : PRUNE_NONE;
    float2 a[8][4];                                  // a[n2][k1]
#pragma unroll
    for (int n2 = 0; n2 < 8; ++n2) {
        a[n2][0] = x[n2]; a[n2][1] = x[n2 + 8]; a[n2][2] = x[n2 + 16]; a[n2][3] = x[n2 + 24];
        dft4<INV, PIN>(a[n2][0], a[n2][1], a[n2][2], a[n2][3]);
    }
    auto column = [&](auto k1c) {
        constexpr int k1 = decltype(k1c)::value;
        float2 c[8];
#pragma unroll
        for (int n2 = 0; n2 < 8; ++n2) c[n2] = a[n2][k1];
        dft8_tw<INV, POUT, k1>(c);                  // the twiddles W32^(n2*k1) are applied inside
#pragma unroll
        for (int k2 = 0; k2 < (PR == PRUNE_OUT ? 4 : 8); ++k2) x[k1 + 4 * k2] = c[k2];
    };
    column(std::integral_constant<int, 0>{}); column(std::integral_constant<int, 1>{});
    column(std::integral_constant<int, 2>{}); column(std::integral_constant<int, 3>{});
}

template <int R, bool INV, int PR> __device__ __forceinline__ void dft(float2 (&x)[R])
{
    if constexpr (R == 2) dft2<INV, PR>(x[0], x[1]);
    else if constexpr (R == 4) dft4<INV, PR>(x[0], x[1], x[2], x[3]);
    else if constexpr (R == 8) dft8<INV, PR>(x);
    else if constexpr (R == 16) dft16<INV, PR>(x);
    else dft32<INV, PR>(x);
}

// ---- pass plan: log2(N) split as evenly as possible into passes of <= 4 bits ------

__host__ __device__ constexpr int n_passes(int log2n) { return (log2n + 3) / 4; }
__host__ __device__ constexpr int pass_bits(int log2n, int s)
{
    const int np = n_passes(log2n);
    return np == 0 ? 0 : log2n / np + (s < log2n % np ? 1 : 0);
}
__host__ __device__ constexpr int bits_before(int log2n, int s)
{
    int b = 0;
    for (int i = 0; i < s; ++i) b += pass_bits(log2n, i);
    return b;
}

// Twiddle table in shared memory: tw[t] = exp(-2 pi i t / N), t in [0, N/2).
template <int N, bool INV> __device__ __forceinline__ float2 twiddle(const float2 *tw, int t)
{
    // t in [0, N)
    float2 w = tw[t & (N / 2 - 1)];
    if (t & (N / 2)) { w.x = -w.x; w.y = -w.y; }
    if (INV) w.y = -w.y;
    return w;
}

// One Stockham pass for item j (0 <= j < N/R) of one line: load + twiddle + DFT.
template <int N, int R, int NS, bool INV, int PR>
__device__ __forceinline__ void pass_load(const float2 *line, int j, const float2 *tw, float2 (&x)[R])
{
    constexpr int NIN = (PR == PRUNE_IN) ? R / 2 : R;
#pragma unroll
    for (int r = 0; r < NIN; ++r) x[r] = line[phys(j + r * (N / R))];
#pragma unroll
    for (int r = NIN; r < R; ++r) x[r] = make_float2(0.f, 0.f);
    if constexpr (NS > 1) {
        const int k = j & (NS - 1);
#pragma unroll
        for (int r = 1; r < NIN; ++r)
            x[r] = cmul(x[r], twiddle<N, INV>(tw, r * k * (N / (NS * R))));
    }
    dft<R, INV, PR>(x);
}

template <int N, int R, int NS, int PR>
__device__ __forceinline__ void pass_store(float2 *line, int j, const float2 (&x)[R])
{
    constexpr int NOUT = (PR == PRUNE_OUT) ? R / 2 : R;
    const int k = j & (NS - 1);
    const int base = (j - k) * R + k;
#pragma unroll
    for (int r = 0; r < NOUT; ++r) line[phys(base + r * NS)] = x[r];
}

// All T threads of the CTA transform G lines (line g at buf + g*LS) in place.
// Ends with a __syncthreads(); callers must have synchronised after filling buf.
template <int LOG2N, bool INV, int PRUNE, int T, int S = 0>
__device__ __forceinline__ void fft_lines(float2 *buf, int G, int LS, const float2 *tw, int tid)
{
    constexpr int N = 1 << LOG2N;
    constexpr int NP = n_passes(LOG2N);
    if constexpr (S < NP) {
        constexpr int R = 1 << pass_bits(LOG2N, S);
        constexpr int NS = 1 << bits_before(LOG2N, S);
        constexpr int PR = (PRUNE == PRUNE_IN && S == 0) ? PRUNE_IN
                         : (PRUNE == PRUNE_OUT && S == NP - 1) ? PRUNE_OUT : PRUNE_NONE;
        constexpr int IPL = N / R;                         // items per line
        if constexpr (IPL <= T) {
            constexpr int LPR = T / IPL;                   // lines per round
            const int gl = tid / IPL, j = tid % IPL;
            for (int g0 = 0; g0 < G; g0 += LPR) {
                const int g = g0 + gl;
                float2 x[R];
                if (g < G) pass_load<N, R, NS, INV, PR>(buf + g * LS, j, tw, x);
                __syncthreads();
                if (g < G) pass_store<N, R, NS, PR>(buf + g * LS, j, x);
            }
        } else {
            constexpr int IT = IPL / T;                    // items per thread per line
            for (int g = 0; g < G; ++g) {
                float2 x[IT][R];
#pragma unroll
                for (int i = 0; i < IT; ++i) pass_load<N, R, NS, INV, PR>(buf + g * LS, tid + i * T, tw, x[i]);
                __syncthreads();
#pragma unroll
                for (int i = 0; i < IT; ++i) pass_store<N, R, NS, PR>(buf + g * LS, tid + i * T, x[i]);
            }
        }
        __syncthreads();
        fft_lines<LOG2N, INV, PRUNE, T, S + 1>(buf, G, LS, tw, tid);
    }
}

// Fill the half twiddle table for N points from a global table of NT >= N points
// (gt[t] = exp(-2 pi i t / NT)); caller synchronises afterwards.
__device__ __forceinline__ void load_twiddles(float2 *tw, const float2 *gt, int N, int NT, int tid, int T)
{
    const int step = NT / N;
    for (int t = tid; t < N / 2; t += T) { HN_G(gt + t * step, 8); tw[t] = gt[t * step]; }
}

}  // namespace hn
