// Contiguous-axis passes of the N-D path, warp-engine version (padded row length 64..1024).
//
//   rows_fwd_w   one group of lanes per pair of rows: the rows are fetched with 16-byte
//                asynchronous copies into the group's line, gated (k*v) and zero-padded on the
//                fly, transformed as one complex row (real part / imaginary part), separated
//                with the Hermitian symmetry and stored as P/2+1 bins per row.
//   rows_inv_w   the inverse: two half spectra are merged into one complex row, transformed
//                back keeping the cropped half, multiplied by q and stored.
#include "common.cuh"
#include "plane_util.cuh"

namespace hn {

constexpr int kRowThreads = 256;

// MODE 0: k*v rows (upper half zero), 1: filter rows with wrapped placement, 2: causal filter rows,
// 3: circular mode, rows of exactly P elements (k*v when b is given, else the filter): power-of-two, aligned rows
// that are read straight from global memory (no staging of misaligned odd-length rows is needed)
// One lane asks the memory system to bring [lo, hi) of an array into L2, trimmed inwards to 16-byte granules.
__device__ __forceinline__ void prefetch_rows_l2(const unsigned char *lo, const unsigned char *hi)
{
    const unsigned long long a0 = ((unsigned long long)lo + 15ull) & ~15ull, a1 = (unsigned long long)hi & ~15ull;
    if (a1 > a0) HN_G((const void *)a0, a1 - a0);
    if (a1 > a0) asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;\n" ::"l"(a0), "r"((unsigned)(a1 - a0)) : "memory");
}

template <typename T, int LOG2P, int MODE>
__global__ void __launch_bounds__(kRowThreads, 2) rows_fwd_w_kernel(RowsArgs p)
{
    using F = WF<LOG2P, false>;
    constexpr int P = 1 << LOG2P, HP = P / 2, TPL = F::TPL, G = kRowThreads / TPL, LS = plane_ls(P);
    constexpr int PR = (MODE == 1 || MODE == 3) ? PRUNE_NONE : PRUNE_IN;
    constexpr int NT = MODE == 0 ? 2 : 1;                                       // tensors per row
    constexpr int ROWMAX = (MODE == 1 ? P - 1 : HP) * (int)sizeof(T);           // longest row in bytes
    constexpr int SLOT = (ROWMAX + 15) / 16 * 16 + 16;
    static_assert(2 * NT * SLOT <= LS * 8, "staged rows must fit the line");
    extern __shared__ float2 smem[];
    float2 *twt = smem + G * LS;
    const int tid = threadIdx.x, l = tid % TPL, gid = tid / TPL;
    const unsigned m = F::group_mask(tid);
    float2 *line = smem + gid * LS;
    for (int t = tid; t < P; t += kRowThreads) { HN_G(p.gtw + t * (p.gtw_n >> LOG2P), 8); twt[t] = p.gtw[t * (p.gtw_n >> LOG2P)]; }
    __syncthreads();
    PlaneTw<LOG2P, false> tw;
    tw.init(l, twt, twt + P, tid, kRowThreads);
    __syncthreads();
    const unsigned char *ab = (const unsigned char *)p.a, *bb = (const unsigned char *)p.b;
    const unsigned char *ahi = ab + p.rows * (long long)p.len * sizeof(T);
    const unsigned char *bhi = bb + p.rows * (long long)p.len * sizeof(T);
    const long long pairs = (p.rows + 1) / 2;
    const int rowb = p.len * (int)sizeof(T);
    for (long long rp = (long long)blockIdx.x * G + gid; rp < pairs; rp += (long long)gridDim.x * G) {
        const long long r0 = 2 * rp, r1 = r0 + 1;
        const bool has1 = r1 < p.rows;
        if constexpr (MODE == 3) {
            const T *a0 = (const T *)p.a + r0 * P, *a1 = (const T *)p.a + (has1 ? r1 : r0) * P;
            const T *b0 = (const T *)p.b + r0 * P, *b1 = (const T *)p.b + (has1 ? r1 : r0) * P;
            const bool gated = p.b != nullptr;
            const float keep1 = has1 ? 1.f : 0.f;
            F::template run_to_line<PR, false>(l, m, tw, line, [&](int, int, int idx) {
                float a = IO<T>::ld(a0, idx), b = IO<T>::ld(a1, idx) * keep1;
                if (gated) { a *= IO<T>::ld(b0, idx); b *= IO<T>::ld(b1, idx); }
                return make_float2(a, b);
            });
            float2 *o0 = p.out + r0 * p.pitch, *o1 = p.out + r1 * p.pitch;
            for (int kx = l; kx <= HP; kx += TPL) {
                const float2 z1 = line[F::ph(kx)], z2 = line[F::ph((P - kx) & (P - 1))];
                HN_G(o0 + kx, 8);
                if (has1) HN_G(o1 + kx, 8);
                o0[kx] = make_float2(0.5f * (z1.x + z2.x), 0.5f * (z1.y - z2.y));
                if (has1) o1[kx] = make_float2(0.5f * (z1.y + z2.y), 0.5f * (z2.x - z1.x));
            }
            __syncwarp(m);
            continue;
        }
        unsigned char *s = reinterpret_cast<unsigned char *>(line);
        const unsigned char *g0 = ab + r0 * rowb, *g1 = ab + r1 * rowb;
        stage_row_u<TPL, ROWMAX>(s, g0, rowb, ab, ahi, l);
        if (has1) stage_row_u<TPL, ROWMAX>(s + SLOT, g1, rowb, ab, ahi, l);
        int fb0 = 0, fb1 = 0;
        if (MODE == 0) {
            const unsigned char *h0 = bb + r0 * rowb, *h1 = bb + r1 * rowb;
            stage_row_u<TPL, ROWMAX>(s + 2 * SLOT, h0, rowb, bb, bhi, l);
            if (has1) stage_row_u<TPL, ROWMAX>(s + 3 * SLOT, h1, rowb, bb, bhi, l);
            fb0 = (int)((unsigned long long)h0 & 15ull);
            fb1 = (int)((unsigned long long)h1 & 15ull);
        }
        if (MODE != 1 && l == 0) {
            // the k and v rows this group takes next travel to L2 while it works on these (measured: a gain for
            // the short k*v rows, none for the long filter rows)
            const long long rn = 2 * (rp + (long long)gridDim.x * G);
            if (rn + 1 < p.rows) {
                prefetch_rows_l2(ab + rn * rowb, ab + (rn + 2) * rowb);
                if (MODE == 0) prefetch_rows_l2(bb + rn * rowb, bb + (rn + 2) * rowb);
            }
        }
        cp_async_wait_all();
        __syncwarp(m);
        const int f0 = (int)((unsigned long long)g0 & 15ull), f1 = (int)((unsigned long long)g1 & 15ull);
        if (MODE == 1) {
            // filter rows: blank the padding taps (and a missing second row) once, then no bounds tests
            zero_staged<T, TPL>(s, f0, p.len, P, l);
            zero_staged<T, TPL>(s + SLOT, f1, has1 ? p.len : 0, P, l);
            __syncwarp(m);
            const int cw = (l + p.shift) & (P - 1);
            F::template run_to_line<PR, true>(l, m, tw, line, [&](int i, int r, int) {
                const int mm = (cw + i * TPL + r * (P / F::template Pass<0>::R)) & (P - 1);
                return make_float2(staged<T>(s, f0, mm), staged<T>(s + SLOT, f1, mm));
            });
        } else if (p.len == HP && has1) {
            // full rows: no bounds tests in the input functor
            F::template run_to_line<PR, true>(l, m, tw, line, [&](int, int, int idx) {
                float a = staged<T>(s, f0, idx), b = staged<T>(s + SLOT, f1, idx);
                if (MODE == 0) {
                    a *= staged<T>(s + 2 * SLOT, fb0, idx);
                    b *= staged<T>(s + 3 * SLOT, fb1, idx);
                }
                return make_float2(a, b);
            });
        } else {
            F::template run_to_line<PR, true>(l, m, tw, line, [&](int, int, int idx) {
                float a = 0.f, b = 0.f;
                if (idx < p.len) {
                    a = staged<T>(s, f0, idx);
                    if (has1) b = staged<T>(s + SLOT, f1, idx);
                    if (MODE == 0) {
                        a *= staged<T>(s + 2 * SLOT, fb0, idx);
                        if (has1) b *= staged<T>(s + 3 * SLOT, fb1, idx);
                    }
                }
                return make_float2(a, b);
            });
        }
        float2 *o0 = p.out + r0 * p.pitch, *o1 = p.out + r1 * p.pitch;
        for (int kx = l; kx <= HP; kx += TPL) {
            const float2 z1 = line[F::ph(kx)], z2 = line[F::ph((P - kx) & (P - 1))];
            HN_G(o0 + kx, 8);
            if (has1) HN_G(o1 + kx, 8);
            o0[kx] = make_float2(0.5f * (z1.x + z2.x), 0.5f * (z1.y - z2.y));
            if (has1) o1[kx] = make_float2(0.5f * (z1.y + z2.y), 0.5f * (z2.x - z1.x));
        }
        __syncwarp(m);
    }
}

// FULL (circular mode): all P outputs of a row are kept.
template <typename T, int LOG2P, bool FULL>
__global__ void __launch_bounds__(kRowThreads, 2) rows_inv_w_kernel(RowsInvArgs p)
{
    using FI = WF<LOG2P, true>;
    constexpr int P = 1 << LOG2P, HP = P / 2, TPL = FI::TPL, G = kRowThreads / TPL, LS = plane_ls(P);
    constexpr int RS = HP + 2;                                   // slot of one staged half spectrum
    static_assert(2 * RS <= LS, "staged spectra must fit the line");
    extern __shared__ float2 smem[];
    float2 *twt = smem + G * LS;
    const int tid = threadIdx.x, l = tid % TPL, gid = tid / TPL;
    const unsigned m = FI::group_mask(tid);
    float2 *line = smem + gid * LS;
    for (int t = tid; t < P; t += kRowThreads) { HN_G(p.gtw + t * (p.gtw_n >> LOG2P), 8); twt[t] = p.gtw[t * (p.gtw_n >> LOG2P)]; }
    __syncthreads();
    PlaneTw<LOG2P, true> tw;
    tw.init(l, twt, twt + P, tid, kRowThreads);
    __syncthreads();
    const T *pq = (const T *)p.q;
    T *py = (T *)p.y;
    const long long pairs = (p.rows + 1) / 2;
    for (long long rp = (long long)blockIdx.x * G + gid; rp < pairs; rp += (long long)gridDim.x * G) {
        const long long r0 = 2 * rp, r1 = r0 + 1;
        const bool has1 = r1 < p.rows;
        const float2 *i0 = p.in + r0 * p.pitch, *i1 = p.in + r1 * p.pitch;
        // rows of the workspace start on 16-byte boundaries (even pitch): two bins per copy
        for (int c = l; 2 * c <= HP; c += TPL) {
            cp_async16(line + 2 * c, i0 + 2 * c);
            if (has1) cp_async16(line + RS + 2 * c, i1 + 2 * c);
        }
        if (!FULL && p.len == HP && has1 && l == 0 && pq) {
            // the two gate rows of the pair (contiguous, a multiple of 16 bytes from a 16-byte boundary)
            const unsigned long long qa = (unsigned long long)(pq + r0 * HP);
            HN_G((const void *)qa, 2 * HP * sizeof(T));
            asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;\n" ::"l"(qa), "r"((unsigned)(2 * HP * sizeof(T))) : "memory");
        }
        cp_async_wait_all();
        __syncwarp(m);
        // Legs below half the first-pass radix read bins <= P/2 directly; the others read the mirrored bin
        // conjugated.  Which case applies is known per leg at compile time, except for the leg that starts at
        // P/2 (its first position is the unmirrored bin P/2 itself).
        if (!has1) for (int c = l; c <= HP; c += TPL) line[RS + c] = make_float2(0.f, 0.f);
        __syncwarp(m);
        constexpr int RH = FI::template Pass<0>::R / 2;
        FI::template run_to_line<FULL ? PRUNE_NONE : PRUNE_OUT, true>(l, m, tw, line, [&](int, int r, int idx) {
            if (r < RH) {
                const float2 A = line[idx], B = line[RS + idx];
                return make_float2(A.x - B.y, A.y + B.x);
            }
            const float2 A = line[P - idx], B = line[RS + P - idx];
            const float sg = (r == RH && idx == HP) ? 1.f : -1.f;
            return make_float2(fmaf(-sg, B.y, A.x), fmaf(sg, A.y, B.x));
        });
        if (!FULL && p.len == HP && has1 && pq) {
            // full rows: all gate loads of the pair are in flight together (they were asked into L2 above)
            float qa[HP / TPL], qb[HP / TPL];
#pragma unroll
            for (int t = 0; t < HP / TPL; ++t) {
                qa[t] = IO<T>::ld(pq, r0 * HP + l + t * TPL);
                qb[t] = IO<T>::ld(pq, r1 * HP + l + t * TPL);
            }
#pragma unroll
            for (int t = 0; t < HP / TPL; ++t) {
                const float2 z = line[FI::ph(l + t * TPL)];
                IO<T>::st(py, r0 * HP + l + t * TPL, z.x * qa[t]);
                IO<T>::st(py, r1 * HP + l + t * TPL, z.y * qb[t]);
            }
        } else {
            if (pq) {
                // (a loop of its own: the read-only gate loads of several iterations go out together)
                for (int n = l; n < p.len; n += TPL) {
                    const float2 z = line[FI::ph(n)];
                    IO<T>::st(py, r0 * p.len + n, z.x * IO<T>::ld(pq, r0 * p.len + n));
                    if (has1) IO<T>::st(py, r1 * p.len + n, z.y * IO<T>::ld(pq, r1 * p.len + n));
                }
            } else {
                // no gate tensor: the rows leave as they are
                for (int n = l; n < p.len; n += TPL) {
                    const float2 z = line[FI::ph(n)];
                    IO<T>::st(py, r0 * p.len + n, z.x);
                    if (has1) IO<T>::st(py, r1 * p.len + n, z.y);
                }
            }
        }
        if (p.y2) {
            // second gate and result: the rows are still in the line
            const T *pq2 = (const T *)p.q2;
            T *py2 = (T *)p.y2;
            for (int n = l; n < p.len; n += TPL) {
                const float2 z = line[FI::ph(n)];
                IO<T>::st(py2, r0 * p.len + n, z.x * IO<T>::ld(pq2, r0 * p.len + n));
                if (has1) IO<T>::st(py2, r1 * p.len + n, z.y * IO<T>::ld(pq2, r1 * p.len + n));
            }
        }
        __syncwarp(m);
    }
}

static int rows_sms()
{
    static int n = 0;
    if (!n) {
        int dev = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
        if (n <= 0) n = 148;
    }
    return n;
}

bool rows_w_supported(int log2p) { return log2p >= 6 && log2p <= 10; }

template <typename T, int LOG2P> static int launch_rows_fwd_w_t(const RowsArgs &a, cudaStream_t st)
{
    using F = WF<LOG2P, false>;
    constexpr int P = 1 << LOG2P, G = kRowThreads / F::TPL, LS = plane_ls(P);
    const size_t sm = sizeof(float2) * ((size_t)G * LS + 2 * P);
    const long long want = ((a.rows + 1) / 2 + G - 1) / G;
    const int grid = (int)(want < 2ll * rows_sms() ? want : 2ll * rows_sms());
    if (grid <= 0) return 0;
#define HN_LAUNCH(MODE)                                                                                  \
    do {                                                                                                 \
        static DevOnce attr;                                                                        \
        if (attr.first()) {                                                                                     \
            cudaFuncSetAttribute(rows_fwd_w_kernel<T, LOG2P, MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm); \
        }                                                                                                \
        rows_fwd_w_kernel<T, LOG2P, MODE><<<grid, kRowThreads, sm, st>>>(a);                             \
    } while (0)
    if (a.full_in) HN_LAUNCH(3);
    else if (a.b) HN_LAUNCH(0);
    else if (a.prune_in) HN_LAUNCH(2);
    else HN_LAUNCH(1);
#undef HN_LAUNCH
    return 1;
}

template <typename T, int LOG2P> static int launch_rows_inv_w_t(const RowsInvArgs &a, cudaStream_t st)
{
    using F = WF<LOG2P, true>;
    constexpr int P = 1 << LOG2P, G = kRowThreads / F::TPL, LS = plane_ls(P);
    const size_t sm = sizeof(float2) * ((size_t)G * LS + 2 * P);
    const long long want = ((a.rows + 1) / 2 + G - 1) / G;
    const int grid = (int)(want < 2ll * rows_sms() ? want : 2ll * rows_sms());
    if (grid <= 0) return 0;
    static DevOnce attr[2];
    void (*fn)(RowsInvArgs) = a.full_out ? rows_inv_w_kernel<T, LOG2P, true> : rows_inv_w_kernel<T, LOG2P, false>;
    if (attr[a.full_out ? 1 : 0].first()) cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
    fn<<<grid, kRowThreads, sm, st>>>(a);
    return 1;
}

#define HN_SWITCH_RW(x, CALL)                                                                  \
    switch (x) {                                                                               \
    case 6: CALL(6); break; case 7: CALL(7); break; case 8: CALL(8); break;                    \
    case 9: CALL(9); break; case 10: CALL(10); break;                                          \
    default: return -1;                                                                        \
    }

int launch_rows_fwd_w(const RowsArgs &a, int dtype, cudaStream_t st)
{
    int n = 0;
#define CALLF(L) n = launch_rows_fwd_w_t<float, L>(a, st)
#define CALLB(L) n = launch_rows_fwd_w_t<bf16, L>(a, st)
    if (dtype == 0) { HN_SWITCH_RW(a.log2p, CALLF) } else { HN_SWITCH_RW(a.log2p, CALLB) }
#undef CALLF
#undef CALLB
    return n;
}

int launch_rows_inv_w(const RowsInvArgs &a, int dtype, cudaStream_t st)
{
    int n = 0;
#define CALLF(L) n = launch_rows_inv_w_t<float, L>(a, st)
#define CALLB(L) n = launch_rows_inv_w_t<bf16, L>(a, st)
    if (dtype == 0) { HN_SWITCH_RW(a.log2p, CALLF) } else { HN_SWITCH_RW(a.log2p, CALLB) }
#undef CALLF
#undef CALLB
    return n;
}

}  // namespace hn
