// Generic N-D path: works for every grid shape the library accepts.
//
//   rows_fwd   gate (k*v), zero-pad and real-to-complex transform along the
//              contiguous axis.  Two real rows ride in one complex transform
//              (real part / imaginary part) and are separated afterwards with
//              the Hermitian symmetry of real-input spectra, so only P/2+1
//              bins per row are kept (half spectrum of Appendix B.1, Eq. 11, 13).
//   axis       complex transforms along a strided axis on tiles of adjacent
//              bins (coalesced loads, lines transposed into shared memory).
//              AXIS_CORE fuses the last forward axis of k*v and of the filter,
//              the spectral product (Eq. 12) and the first inverse axis.
//   rows_inv   complex-to-real inverse along the contiguous axis, crop to the
//              grid, output gate q, store.
#include "common.cuh"
#include "fft_engine.cuh"

namespace hn {

static int g_sm_count = 0;
static int sm_count()
{
    if (!g_sm_count) {
        int dev = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&g_sm_count, cudaDevAttrMultiProcessorCount, dev);
        if (g_sm_count <= 0) g_sm_count = 148;
    }
    return g_sm_count;
}

__host__ __device__ static inline int lines_per_chunk(int log2p)
{
    int g = 4096 >> log2p;
    return g < 1 ? 1 : (g > 32 ? 32 : g);
}

static size_t smem_bytes(int log2p, int lines, int buffers)
{
    const int n = 1 << log2p;
    return sizeof(float2) * ((size_t)buffers * lines * line_stride(n) + (n >= 2 ? n / 2 : 1));
}

// ---- rows, forward ----------------------------------------------------------------

template <typename T, int LOG2P, bool HAS_B, bool PRUNE>
__global__ void __launch_bounds__(kThreads) rows_fwd_kernel(RowsArgs p)
{
    constexpr int N = 1 << LOG2P;
    constexpr int LS = line_stride(N);
    constexpr int NFILL = PRUNE && N >= 2 ? N / 2 : N;
    constexpr int XH = N / 2 + 1;
    extern __shared__ float2 smem[];
    const int G = lines_per_chunk(LOG2P);
    float2 *buf = smem;
    float2 *tw = smem + G * LS;
    const int tid = threadIdx.x;
    const T *pa = (const T *)p.a;
    const T *pb = (const T *)p.b;
    if (N >= 4) load_twiddles(tw, p.gtw, N, p.gtw_n, tid, kThreads);
    const long long pairs = (p.rows + 1) / 2;
    const long long chunks = (pairs + G - 1) / G;
    for (long long ch = blockIdx.x; ch < chunks; ch += gridDim.x) {
        for (int idx = tid; idx < G * NFILL; idx += kThreads) {
            const int g = idx / NFILL, pos = idx % NFILL;
            const long long r0 = 2 * (ch * G + g), r1 = r0 + 1;
            const int m = (pos + p.shift) & (N - 1);
            float a0 = 0.f, a1 = 0.f;
            if (m < p.len) {
                if (r0 < p.rows) {
                    a0 = IO<T>::ld(pa, r0 * p.len + m);
                    if (HAS_B) a0 *= IO<T>::ld(pb, r0 * p.len + m);
                }
                if (r1 < p.rows) {
                    a1 = IO<T>::ld(pa, r1 * p.len + m);
                    if (HAS_B) a1 *= IO<T>::ld(pb, r1 * p.len + m);
                }
            }
            buf[g * LS + phys(pos)] = make_float2(a0, a1);
        }
        __syncthreads();
        fft_lines<LOG2P, false, PRUNE ? PRUNE_IN : PRUNE_NONE, kThreads>(buf, G, LS, tw, tid);
        for (int idx = tid; idx < G * XH; idx += kThreads) {
            const int g = idx / XH, kx = idx % XH;
            const long long r0 = 2 * (ch * G + g), r1 = r0 + 1;
            const float2 z1 = buf[g * LS + phys(kx)];
            const float2 z2 = buf[g * LS + phys((N - kx) & (N - 1))];
            if (r0 < p.rows) { HN_G(p.out + r0 * p.pitch + kx, 8); p.out[r0 * p.pitch + kx] = make_float2(0.5f * (z1.x + z2.x), 0.5f * (z1.y - z2.y)); }
            if (r1 < p.rows) { HN_G(p.out + r1 * p.pitch + kx, 8); p.out[r1 * p.pitch + kx] = make_float2(0.5f * (z1.y + z2.y), 0.5f * (z2.x - z1.x)); }
        }
        __syncthreads();
    }
}

template <typename T, int LOG2P>
static int launch_rows_fwd_t(const RowsArgs &a, cudaStream_t st)
{
    const int G = lines_per_chunk(LOG2P);
    const size_t sm = smem_bytes(LOG2P, G, 1);
    const long long pairs = (a.rows + 1) / 2;
    const long long chunks = (pairs + G - 1) / G;
    const int grid = (int)(chunks < (long long)sm_count() * 8 ? chunks : (long long)sm_count() * 8);
    if (grid <= 0) return 0;
#define HN_LAUNCH(HASB, PR)                                                                     \
    do {                                                                                        \
        static DevOnce attr;                                                               \
        if (attr.first()) {                                                                            \
            cudaFuncSetAttribute(rows_fwd_kernel<T, LOG2P, HASB, PR>,                           \
                                 cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);         \
        }                                                                                       \
        rows_fwd_kernel<T, LOG2P, HASB, PR><<<grid, kThreads, sm, st>>>(a);                     \
    } while (0)
    if (a.b && a.full_in) HN_LAUNCH(true, false);
    else if (a.b) HN_LAUNCH(true, true);
    else if (a.prune_in) HN_LAUNCH(false, true);
    else HN_LAUNCH(false, false);
#undef HN_LAUNCH
    return 1;
}

#define HN_SWITCH_LOG2P(x, CALL)                                                                \
    switch (x) {                                                                                \
    case 0: CALL(0); break; case 1: CALL(1); break; case 2: CALL(2); break;                     \
    case 3: CALL(3); break; case 4: CALL(4); break; case 5: CALL(5); break;                     \
    case 6: CALL(6); break; case 7: CALL(7); break; case 8: CALL(8); break;                     \
    case 9: CALL(9); break; case 10: CALL(10); break; case 11: CALL(11); break;                 \
    case 12: CALL(12); break; case 13: CALL(13); break;                                         \
    default: return -1;                                                                         \
    }

int launch_rows_fwd(const RowsArgs &a, int dtype, cudaStream_t st)
{
    int n = 0;
#define CALLF(L) n = launch_rows_fwd_t<float, L>(a, st)
#define CALLB(L) n = launch_rows_fwd_t<bf16, L>(a, st)
    if (dtype == 0) { HN_SWITCH_LOG2P(a.log2p, CALLF) } else { HN_SWITCH_LOG2P(a.log2p, CALLB) }
#undef CALLF
#undef CALLB
    return n;
}

// ---- rows, inverse + crop + output gate ----------------------------------------------

template <typename T, int LOG2P, bool FULL>
__global__ void __launch_bounds__(kThreads) rows_inv_kernel(RowsInvArgs p)
{
    constexpr int N = 1 << LOG2P;
    constexpr int LS = line_stride(N);
    extern __shared__ float2 smem[];
    const int G = lines_per_chunk(LOG2P);
    float2 *buf = smem;
    float2 *tw = smem + G * LS;
    const int tid = threadIdx.x;
    const T *pq = (const T *)p.q;
    T *py = (T *)p.y;
    if (N >= 4) load_twiddles(tw, p.gtw, N, p.gtw_n, tid, kThreads);
    const long long pairs = (p.rows + 1) / 2;
    const long long chunks = (pairs + G - 1) / G;
    for (long long ch = blockIdx.x; ch < chunks; ch += gridDim.x) {
        for (int idx = tid; idx < G * N; idx += kThreads) {
            const int g = idx / N, pos = idx % N;
            const long long r0 = 2 * (ch * G + g), r1 = r0 + 1;
            const bool mirror = pos > N / 2;
            const int kx = mirror ? N - pos : pos;
            float2 A = make_float2(0.f, 0.f), B = A;
            if (r0 < p.rows) { HN_G(p.in + r0 * p.pitch + kx, 8); A = p.in[r0 * p.pitch + kx]; }
            if (r1 < p.rows) { HN_G(p.in + r1 * p.pitch + kx, 8); B = p.in[r1 * p.pitch + kx]; }
            if (mirror) { A.y = -A.y; B.y = -B.y; }
            buf[g * LS + phys(pos)] = make_float2(A.x - B.y, A.y + B.x);
        }
        __syncthreads();
        fft_lines<LOG2P, true, FULL ? PRUNE_NONE : PRUNE_OUT, kThreads>(buf, G, LS, tw, tid);
        if (pq) {
            for (int idx = tid; idx < G * p.len; idx += kThreads) {
                const int g = idx / p.len, n = idx % p.len;
                const long long r0 = 2 * (ch * G + g), r1 = r0 + 1;
                const float2 z = buf[g * LS + phys(n)];
                if (r0 < p.rows) IO<T>::st(py, r0 * p.len + n, z.x * IO<T>::ld(pq, r0 * p.len + n));
                if (r1 < p.rows) IO<T>::st(py, r1 * p.len + n, z.y * IO<T>::ld(pq, r1 * p.len + n));
            }
        } else {
            // no gate tensor: the rows leave as they are
            for (int idx = tid; idx < G * p.len; idx += kThreads) {
                const int g = idx / p.len, n = idx % p.len;
                const long long r0 = 2 * (ch * G + g), r1 = r0 + 1;
                const float2 z = buf[g * LS + phys(n)];
                if (r0 < p.rows) IO<T>::st(py, r0 * p.len + n, z.x);
                if (r1 < p.rows) IO<T>::st(py, r1 * p.len + n, z.y);
            }
        }
        if (p.y2) {
            // second gate and result: the rows are still in the buffer
            const T *pq2 = (const T *)p.q2;
            T *py2 = (T *)p.y2;
            for (int idx = tid; idx < G * p.len; idx += kThreads) {
                const int g = idx / p.len, n = idx % p.len;
                const long long r0 = 2 * (ch * G + g), r1 = r0 + 1;
                const float2 z = buf[g * LS + phys(n)];
                if (r0 < p.rows) IO<T>::st(py2, r0 * p.len + n, z.x * IO<T>::ld(pq2, r0 * p.len + n));
                if (r1 < p.rows) IO<T>::st(py2, r1 * p.len + n, z.y * IO<T>::ld(pq2, r1 * p.len + n));
            }
        }
        __syncthreads();
    }
}

template <typename T, int LOG2P>
static int launch_rows_inv_t(const RowsInvArgs &a, cudaStream_t st)
{
    const int G = lines_per_chunk(LOG2P);
    const size_t sm = smem_bytes(LOG2P, G, 1);
    const long long pairs = (a.rows + 1) / 2;
    const long long chunks = (pairs + G - 1) / G;
    const int grid = (int)(chunks < (long long)sm_count() * 8 ? chunks : (long long)sm_count() * 8);
    if (grid <= 0) return 0;
    static DevOnce attr[2];
    void (*fn)(RowsInvArgs) = a.full_out ? rows_inv_kernel<T, LOG2P, true> : rows_inv_kernel<T, LOG2P, false>;
    if (attr[a.full_out ? 1 : 0].first()) cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
    fn<<<grid, kThreads, sm, st>>>(a);
    return 1;
}

int launch_rows_inv(const RowsInvArgs &a, int dtype, cudaStream_t st)
{
    int n = 0;
#define CALLF(L) n = launch_rows_inv_t<float, L>(a, st)
#define CALLB(L) n = launch_rows_inv_t<bf16, L>(a, st)
    if (dtype == 0) { HN_SWITCH_LOG2P(a.log2p, CALLF) } else { HN_SWITCH_LOG2P(a.log2p, CALLB) }
#undef CALLF
#undef CALLB
    return n;
}

// ---- strided axes -----------------------------------------------------------------------

// Fill TX lines of one tile: element m of line x comes from src[m*nc + x], goes to
// position (m - shift) mod N.  Threads run along x first (coalesced).
template <int N, int NFILL>
__device__ __forceinline__ void fill_tile(float2 *buf, int LS, int TX, const float2 *src, int nc, int width,
                                          int n_in, int shift, int tid)
{
    for (int idx = tid; idx < TX * NFILL; idx += kThreads) {
        const int x = idx % TX, pos = idx / TX;
        const int m = (pos + shift) & (N - 1);
        float2 val = make_float2(0.f, 0.f);
        if (m < n_in && x < width) { HN_G(src + (long long)m * nc + x, 8); val = src[(long long)m * nc + x]; }
        buf[x * LS + phys(pos)] = val;
    }
}

template <int MODE, int LOG2P, bool PRUNE>
__global__ void __launch_bounds__(kThreads) axis_kernel(AxisArgs p)
{
    constexpr int N = 1 << LOG2P;
    constexpr int LS = line_stride(N);
    constexpr int NFILL_U = (MODE != AXIS_INV && PRUNE && N >= 2) ? N / 2 : N;
    extern __shared__ float2 smem[];
    const int TX = lines_per_chunk(LOG2P);
    float2 *bu = smem;
    float2 *bh = smem + TX * LS;                                   // core only
    float2 *tw = smem + (MODE == AXIS_CORE ? 2 : 1) * TX * LS;
    const int tid = threadIdx.x;
    if (N >= 4) load_twiddles(tw, p.gtw, N, p.gtw_n, tid, kThreads);
    const long long tpo = (p.nc + TX - 1) / TX;
    const long long tiles = p.n_outer * tpo;
    for (long long t = blockIdx.x; t < tiles; t += gridDim.x) {
        const long long o = t / tpo;
        const int c0 = (int)(t % tpo) * TX;
        const int width = p.nc - c0 < TX ? p.nc - c0 : TX;
        fill_tile<N, NFILL_U>(bu, LS, TX, p.in + o * p.in_outer + c0, p.nc, width, p.n_in, p.shift, tid);
        if (MODE == AXIS_CORE) {
            const long long oh = p.h_mod ? (o + p.h_off) % p.h_mod : o;
            fill_tile<N, N>(bh, LS, TX, p.h + oh * p.h_outer + c0, p.nc, width, p.h_n_in, p.h_shift, tid);
        }
        __syncthreads();
        if (MODE == AXIS_INV) {
            fft_lines<LOG2P, true, PRUNE ? PRUNE_OUT : PRUNE_NONE, kThreads>(bu, TX, LS, tw, tid);
        } else {
            fft_lines<LOG2P, false, PRUNE ? PRUNE_IN : PRUNE_NONE, kThreads>(bu, TX, LS, tw, tid);
        }
        if (MODE == AXIS_CORE) {
            fft_lines<LOG2P, false, PRUNE_NONE, kThreads>(bh, TX, LS, tw, tid);
            for (int idx = tid; idx < TX * N; idx += kThreads) {
                const int x = idx / N, pos = idx % N;
                const int a = x * LS + phys(pos);
                float2 w = p.h_conj ? cmulc(bu[a], bh[a]) : cmul(bu[a], bh[a]);
                bu[a] = make_float2(w.x * p.scale, w.y * p.scale);
            }
            __syncthreads();
            fft_lines<LOG2P, true, PRUNE ? PRUNE_OUT : PRUNE_NONE, kThreads>(bu, TX, LS, tw, tid);
        }
        float2 *dst = p.out + o * p.out_outer + c0;
        for (int idx = tid; idx < TX * p.n_out; idx += kThreads) {
            const int x = idx % TX, a = idx / TX;
            if (x < width) { HN_G(dst + (long long)a * p.nc + x, 8); dst[(long long)a * p.nc + x] = bu[x * LS + phys(a)]; }
        }
        __syncthreads();
    }
}

template <int MODE, int LOG2P, bool PRUNE>
static int launch_axis_t(const AxisArgs &a, cudaStream_t st)
{
    const int TX = lines_per_chunk(LOG2P);
    const size_t sm = smem_bytes(LOG2P, TX, MODE == AXIS_CORE ? 2 : 1);
    const long long tiles = a.n_outer * ((a.nc + TX - 1) / TX);
    const int grid = (int)(tiles < (long long)sm_count() * 8 ? tiles : (long long)sm_count() * 8);
    if (grid <= 0) return 0;
    static DevOnce attr;
    if (attr.first()) {
        cudaFuncSetAttribute(axis_kernel<MODE, LOG2P, PRUNE>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
    }
    axis_kernel<MODE, LOG2P, PRUNE><<<grid, kThreads, sm, st>>>(a);
    return 1;
}

int launch_axis(const AxisArgs &a, int mode, cudaStream_t st)
{
    int n = 0;
#define CALL_FP(L) n = launch_axis_t<AXIS_FWD, L, true>(a, st)
#define CALL_FN(L) n = launch_axis_t<AXIS_FWD, L, false>(a, st)
    // inverse and core: the flag selects the cropped (pruned) output half, or the whole line in circular mode
#define CALL_I(L) n = launch_axis_t<AXIS_INV, L, true>(a, st)
#define CALL_IF(L) n = launch_axis_t<AXIS_INV, L, false>(a, st)
#define CALL_C(L) n = launch_axis_t<AXIS_CORE, L, true>(a, st)
#define CALL_CF(L) n = launch_axis_t<AXIS_CORE, L, false>(a, st)
    if (mode == AXIS_FWD && a.prune_in) { HN_SWITCH_LOG2P(a.log2p, CALL_FP) }
    else if (mode == AXIS_FWD) { HN_SWITCH_LOG2P(a.log2p, CALL_FN) }
    else if (mode == AXIS_INV && a.full) { HN_SWITCH_LOG2P(a.log2p, CALL_IF) }
    else if (mode == AXIS_INV) { HN_SWITCH_LOG2P(a.log2p, CALL_I) }
    else if (a.full) { HN_SWITCH_LOG2P(a.log2p, CALL_CF) }
    else { HN_SWITCH_LOG2P(a.log2p, CALL_C) }
#undef CALL_FP
#undef CALL_FN
#undef CALL_I
#undef CALL_IF
#undef CALL_C
#undef CALL_CF
    return n;
}

}  // namespace hn
