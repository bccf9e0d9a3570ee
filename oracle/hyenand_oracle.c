/*
 * CPU oracle for the gated N-D long convolution (TEST INFRASTRUCTURE ONLY).
 *
 * This file is the slow, plain reference that the CUDA library is judged
 * against.  It shares no code with the CUDA path, is never linked into the
 * product library, and must only be called from the tests, the smoke check
 * and the benchmark's CPU-baseline leg.
 *
 * Operator (gated Hyena mixer, Definition A.3 / Eq. 1 of the paper, with the
 * depthwise kernel of Definition A.2): for every batch entry b, channel c and
 * grid position i,
 *
 *     y[b,c,i] = q[b,c,i] * sum_j  K[b,c, i - j] * k[b,c,j] * v[b,c,j]
 *
 * where the weight of input j for output i depends on the displacement i - j
 * only (Toeplitz form, Theorem A.5), q is the output gate and k*v the input
 * gate.  Boundary handling (Section 3.2.1 "circular and non-circular
 * convolutions", Appendix "Masking strategy"):
 *   mode 0  linear, non-causal: the kernel lives on (2L_1-1) x ... x (2L_N-1)
 *           displacements, tap index m_n = (i_n - j_n) + (L_n - 1); inputs are
 *           zero outside the grid, outputs are cropped to the grid.
 *   mode 1  causal (1-D only): negative displacements carry zero weight, the
 *           kernel has L taps, tap index m = i - j >= 0.
 *   mode 2  circular (periodic boundary): the kernel lives on the grid itself,
 *           tap index m_n = (i_n - j_n) mod L_n.
 *
 * Two independent evaluations are provided, everything in fp64:
 *   O1  hn_oracle_direct / hn_oracle_direct_at: the sums above, literally.
 *   O2  hn_oracle_fft: zero-pad to a power-of-two torus P_n >= 2L_n-1 (P_n = L_n
 *       padded up is NOT used for the circular mode, which needs L_n itself a
 *       power of two), full complex radix-2 FFT along every axis, spectral
 *       product, inverse, crop, gate (Appendix B.1, Eq. 11-13).
 * No blocking, pruning or fusion: the code follows the definition step by step.
 *
 * Layout: q,k,v,y are [B][C][L_1]..[L_N] row-major; h is [Bh][C][K_1]..[K_N]
 * with K_n = 2L_n-1 (mode 0), L_1 (mode 1), L_n (mode 2); h_batch_stride is the
 * element distance between consecutive batch entries of h (0 = one kernel per
 * channel shared by the whole batch).
 *
 * Parity pins: every function here is pinned by tests/test_oracle_pins.py
 * (hand-worked examples from the definition, closed forms, library routines,
 * brute force); nothing is "parity unpinned".
 */
#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define HN_MAXD 3

int hn_oracle_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

static long long prod(const int *d, int n)
{
    long long p = 1;
    for (int a = 0; a < n; ++a) p *= d[a];
    return p;
}

static int taps_of(int mode, int L)
{
    return mode == 0 ? 2 * L - 1 : L;
}

/* tap index along one axis for displacement d = i - j, or -1 when the kernel
 * gives that displacement no weight */
static int tap_index(int mode, int L, int d)
{
    if (mode == 0) return d + (L - 1);          /* d in [-(L-1), L-1] */
    if (mode == 1) return d >= 0 ? d : -1;      /* causal: 1[r >= 0] */
    return ((d % L) + L) % L;                   /* circular */
}

/* one output value of the ungated convolution, by the definition */
static double conv_at(int ndim, const int *L, const int *K, int mode,
                      const double *k, const double *v, const double *h,
                      const int *i)
{
    double acc = 0.0;
    int j[HN_MAXD] = {0, 0, 0};
    long long n = prod(L, ndim);
    for (long long f = 0; f < n; ++f) {
        /* unravel f -> j */
        long long r = f;
        for (int a = ndim - 1; a >= 0; --a) { j[a] = (int)(r % L[a]); r /= L[a]; }
        long long hidx = 0;
        int ok = 1;
        for (int a = 0; a < ndim; ++a) {
            int m = tap_index(mode, L[a], i[a] - j[a]);
            if (m < 0) { ok = 0; break; }
            hidx = hidx * K[a] + m;
        }
        if (ok) acc += h[hidx] * (k[f] * v[f]);
    }
    return acc;
}

static int check_args(int ndim, const int *dims, int B, int C, int mode)
{
    if (ndim < 1 || ndim > HN_MAXD || B < 1 || C < 1) return 1;
    if (mode < 0 || mode > 2) return 1;
    if (mode == 1 && ndim != 1) return 2;
    for (int a = 0; a < ndim; ++a) if (dims[a] < 1) return 1;
    return 0;
}

/* O1, whole tensor. */
int hn_oracle_direct(int ndim, const int *dims, int B, int C, int mode,
                     const double *q, const double *k, const double *v,
                     const double *h, long long h_batch_stride, double *y)
{
    int e = check_args(ndim, dims, B, C, mode);
    if (e) return e;
    int K[HN_MAXD];
    for (int a = 0; a < ndim; ++a) K[a] = taps_of(mode, dims[a]);
    long long n = prod(dims, ndim), nk = prod(K, ndim);
    long long total = (long long)B * C * n;
#pragma omp parallel for schedule(static)
    for (long long t = 0; t < total; ++t) {
        long long s = t / n, f = t % n;
        int b = (int)(s / C), c = (int)(s % C);
        int i[HN_MAXD] = {0, 0, 0};
        long long r = f;
        for (int a = ndim - 1; a >= 0; --a) { i[a] = (int)(r % dims[a]); r /= dims[a]; }
        const double *hs = h + (long long)b * h_batch_stride + (long long)c * nk;
        y[t] = q[t] * conv_at(ndim, dims, K, mode, k + s * n, v + s * n, hs, i);
    }
    return 0;
}

/* O1 at chosen output positions: flat[t] indexes the [B][C][L..] tensor. */
int hn_oracle_direct_at(int ndim, const int *dims, int B, int C, int mode,
                        const double *q, const double *k, const double *v,
                        const double *h, long long h_batch_stride,
                        long long count, const long long *flat, double *y_out)
{
    int e = check_args(ndim, dims, B, C, mode);
    if (e) return e;
    int K[HN_MAXD];
    for (int a = 0; a < ndim; ++a) K[a] = taps_of(mode, dims[a]);
    long long n = prod(dims, ndim), nk = prod(K, ndim);
#pragma omp parallel for schedule(dynamic, 1)
    for (long long t = 0; t < count; ++t) {
        long long s = flat[t] / n, f = flat[t] % n;
        int b = (int)(s / C), c = (int)(s % C);
        int i[HN_MAXD] = {0, 0, 0};
        long long r = f;
        for (int a = ndim - 1; a >= 0; --a) { i[a] = (int)(r % dims[a]); r /= dims[a]; }
        const double *hs = h + (long long)b * h_batch_stride + (long long)c * nk;
        y_out[t] = q[flat[t]] * conv_at(ndim, dims, K, mode, k + s * n, v + s * n, hs, i);
    }
    return 0;
}

/* ---- O2: naive radix-2 FFT path ------------------------------------------ */

static int next_pow2(int x)
{
    int p = 1;
    while (p < x) p <<= 1;
    return p;
}

/* In-place iterative radix-2 decimation-in-time FFT on n = 2^m points with
 * stride `st` between consecutive points (interleaved re,im doubles).
 * Forward kernel e^{-2 pi i jk/n}; the inverse uses the conjugate kernel and
 * leaves the 1/n factor to the caller.  Twiddles come from cos/sin of each
 * index, never from a recurrence. */
static void fft_line(double *x, long long st, int n, int inverse)
{
    /* bit reversal permutation */
    for (int i = 1, j = 0; i < n; ++i) {
        int bit = n >> 1;
        for (; j & bit; bit >>= 1) j ^= bit;
        j ^= bit;
        if (i < j) {
            double tr = x[2 * i * st], ti = x[2 * i * st + 1];
            x[2 * i * st] = x[2 * j * st]; x[2 * i * st + 1] = x[2 * j * st + 1];
            x[2 * j * st] = tr; x[2 * j * st + 1] = ti;
        }
    }
    const double sgn = inverse ? 1.0 : -1.0;
    for (int len = 2; len <= n; len <<= 1) {
        int half = len >> 1;
        for (int start = 0; start < n; start += len) {
            for (int t = 0; t < half; ++t) {
                double ang = sgn * 2.0 * M_PI * (double)t / (double)len;
                double wr = cos(ang), wi = sin(ang);
                double *a = x + 2 * (long long)(start + t) * st;
                double *b = x + 2 * (long long)(start + t + half) * st;
                double br = b[0] * wr - b[1] * wi;
                double bi = b[0] * wi + b[1] * wr;
                b[0] = a[0] - br; b[1] = a[1] - bi;
                a[0] += br;       a[1] += bi;
            }
        }
    }
}

/* N-D complex transform of a [P_1]..[P_N] row-major array (interleaved), one
 * axis after the other.  Every P_n must be a power of two.  Unnormalised. */
int hn_oracle_fftn(int ndim, const int *P, double *x, int inverse)
{
    if (ndim < 1 || ndim > HN_MAXD) return 1;
    for (int a = 0; a < ndim; ++a) if (P[a] < 1 || (P[a] & (P[a] - 1))) return 1;
    long long total = prod(P, ndim);
    long long stride = 1;
    for (int a = ndim - 1; a >= 0; --a) {
        long long lines = total / P[a];
        for (long long ln = 0; ln < lines; ++ln) {
            /* line ln: all indices with the a-th coordinate free */
            long long inner = ln % stride, outer = ln / stride;
            long long base = outer * stride * P[a] + inner;
            fft_line(x + 2 * base, stride, P[a], inverse);
        }
        stride *= P[a];
    }
    return 0;
}

/* Place a real [n_1]..[n_N] array into the zeroed complex torus [P], entry
 * `idx` along axis a going to (idx + shift_a) mod P_a. */
static void scatter_real(int ndim, const int *n, const int *P, const int *shift,
                         const double *src, double *dst)
{
    long long cnt = prod(n, ndim);
    for (long long f = 0; f < cnt; ++f) {
        long long r = f, pidx = 0, mul = 1;
        int idx[HN_MAXD];
        for (int a = ndim - 1; a >= 0; --a) { idx[a] = (int)(r % n[a]); r /= n[a]; }
        for (int a = ndim - 1; a >= 0; --a) {
            int p = ((idx[a] + shift[a]) % P[a] + P[a]) % P[a];
            pidx += (long long)p * mul;
            mul *= P[a];
        }
        dst[2 * pidx] = src[f];
    }
}

/* O2, whole tensor. */
int hn_oracle_fft(int ndim, const int *dims, int B, int C, int mode,
                  const double *q, const double *k, const double *v,
                  const double *h, long long h_batch_stride, double *y)
{
    int e = check_args(ndim, dims, B, C, mode);
    if (e) return e;
    int K[HN_MAXD], P[HN_MAXD], hshift[HN_MAXD], zero[HN_MAXD] = {0, 0, 0};
    for (int a = 0; a < ndim; ++a) {
        K[a] = taps_of(mode, dims[a]);
        if (mode == 2) {
            if (dims[a] & (dims[a] - 1)) return 2;   /* radix-2 only */
            P[a] = dims[a];
            hshift[a] = 0;
        } else {
            P[a] = next_pow2(2 * dims[a] - 1);
            /* displacement d sits at torus index d mod P: tap m = d + (L-1) */
            hshift[a] = mode == 0 ? -(dims[a] - 1) : 0;
        }
    }
    long long n = prod(dims, ndim), nk = prod(K, ndim), np = prod(P, ndim);
    long long slices = (long long)B * C;
    int failed = 0;
#pragma omp parallel
    {
        double *U = (double *)malloc(sizeof(double) * 2 * np);
        double *H = (double *)malloc(sizeof(double) * 2 * np);
        double *u = (double *)malloc(sizeof(double) * n);
        if (!U || !H || !u) {
#pragma omp atomic write
            failed = 1;
        } else {
#pragma omp for schedule(dynamic, 1)
            for (long long s = 0; s < slices; ++s) {
                int b = (int)(s / C), c = (int)(s % C);
                const double *hs = h + (long long)b * h_batch_stride + (long long)c * nk;
                for (long long f = 0; f < n; ++f) u[f] = k[s * n + f] * v[s * n + f];
                memset(U, 0, sizeof(double) * 2 * np);
                memset(H, 0, sizeof(double) * 2 * np);
                scatter_real(ndim, dims, P, zero, u, U);
                scatter_real(ndim, K, P, hshift, hs, H);
                hn_oracle_fftn(ndim, P, U, 0);
                hn_oracle_fftn(ndim, P, H, 0);
                for (long long t = 0; t < np; ++t) {
                    double ar = U[2 * t], ai = U[2 * t + 1];
                    double br = H[2 * t], bi = H[2 * t + 1];
                    U[2 * t] = ar * br - ai * bi;
                    U[2 * t + 1] = ar * bi + ai * br;
                }
                hn_oracle_fftn(ndim, P, U, 1);
                /* crop: output i sits at torus index i */
                for (long long f = 0; f < n; ++f) {
                    long long r = f, pidx = 0, mul = 1;
                    for (int a = ndim - 1; a >= 0; --a) {
                        int ia = (int)(r % dims[a]); r /= dims[a];
                        pidx += (long long)ia * mul;
                        mul *= P[a];
                    }
                    y[s * n + f] = q[s * n + f] * (U[2 * pidx] / (double)np);
                }
            }
        }
        free(U); free(H); free(u);
    }
    return failed ? 3 : 0;
}
