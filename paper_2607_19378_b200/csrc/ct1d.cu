// Long 1-D path.  A padded sequence of P = P1*P2 points is viewed as a P1 x P2
// array (time index t = t1*P2 + t2, frequency index f = f1 + P1*f2) and
// transformed in two passes, the decomposition Appendix B.3 of the paper uses
// for sequences beyond one thread block's reach:
//
//   cols_fwd  transform along t1 for every column t2.  Two adjacent real columns
//             ride in one complex transform and are separated with the Hermitian
//             symmetry, so only f1 in [0, P1/2] is kept; each entry is multiplied
//             by the inter-pass twiddle W_P^(t2*f1) and stored as [f1][t2].
//   core      for every kept f1: transform the row along t2 for k*v and for the
//             filter, multiply (Eq. 12), transform back, undo the twiddle.
//   cols_inv  rebuild the mirrored half, inverse transform along f1, keep
//             t < L (crop), apply the output gate q, store.
#include <math.h>
#include <stdlib.h>

#include <vector>

#include "common.cuh"
#include "ct1d.cuh"
#include "fft_engine.cuh"

namespace hn {

static int sms()
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

__host__ __device__ static inline int tile_lines(int log2n)
{
    int g = 4096 >> log2n;
    return g < 1 ? 1 : (g > 32 ? 32 : g);
}

// W_P^j from a coarse and a fine table: j = a * 2^lo + b.
struct TwoLevel {
    const float2 *coarse, *fine;
    int lo;
};
__device__ __forceinline__ float2 twiddle_p(const TwoLevel &t, unsigned j)
{
    HN_G(t.coarse + (j >> t.lo), 8);
    HN_G(t.fine + (j & ((1u << t.lo) - 1)), 8);
    const float2 c = __ldg(t.coarse + (j >> t.lo));
    const float2 f = __ldg(t.fine + (j & ((1u << t.lo) - 1)));
    return cmul(c, f);
}

struct ColsFwdArgs {
    const void *a, *b;      // k, v  (or h, nullptr)
    float2 *out;            // [slices][P1/2+1][P2]
    long long slices;
    long long in_slice;     // elements per slice of the input
    int len;                // valid elements
    int shift;              // element m sits at time (m - shift) mod P
    int log2p2;
    const float2 *tw1; int tw1_n;
    TwoLevel twp;
};

template <typename T, int LOG2P1, bool HAS_B, bool PRUNE>
__global__ void __launch_bounds__(kThreads) ct_cols_fwd_kernel(ColsFwdArgs p)
{
    constexpr int P1 = 1 << LOG2P1;
    constexpr int LS = line_stride(P1);
    constexpr int NFILL = PRUNE ? P1 / 2 : P1;
    constexpr int F1 = P1 / 2 + 1;
    extern __shared__ float2 smem[];
    const int TX = tile_lines(LOG2P1);
    float2 *buf = smem;
    float2 *tw = smem + TX * LS;
    const int tid = threadIdx.x;
    const T *pa = (const T *)p.a;
    const T *pb = (const T *)p.b;
    load_twiddles(tw, p.tw1, P1, p.tw1_n, tid, kThreads);
    const int P2 = 1 << p.log2p2;
    const unsigned Pm = (1u << (LOG2P1 + p.log2p2)) - 1u;
    const int tpc = (P2 / 2 + TX - 1) / TX;                  // tiles of column pairs per slice
    const long long tiles = p.slices * tpc;
    for (long long t = blockIdx.x; t < tiles; t += gridDim.x) {
        const long long s = t / tpc;
        const int c0 = (int)(t % tpc) * TX;
        const int width = P2 / 2 - c0 < TX ? P2 / 2 - c0 : TX;
        const long long base = s * p.in_slice;
        for (int idx = tid; idx < TX * NFILL; idx += kThreads) {
            const int x = idx % TX, t1 = idx / TX;
            float a0 = 0.f, a1 = 0.f;
            if (x < width) {
                const unsigned tt = (unsigned)t1 * P2 + 2u * (c0 + x);
                const unsigned m0 = (tt + p.shift) & Pm, m1 = (tt + 1u + p.shift) & Pm;
                if (m0 < (unsigned)p.len) {
                    a0 = IO<T>::ld(pa, base + m0);
                    if (HAS_B) a0 *= IO<T>::ld(pb, base + m0);
                }
                if (m1 < (unsigned)p.len) {
                    a1 = IO<T>::ld(pa, base + m1);
                    if (HAS_B) a1 *= IO<T>::ld(pb, base + m1);
                }
            }
            buf[x * LS + phys(t1)] = make_float2(a0, a1);
        }
        __syncthreads();
        fft_lines<LOG2P1, false, PRUNE ? PRUNE_IN : PRUNE_NONE, kThreads>(buf, TX, LS, tw, tid);
        float2 *dst = p.out + s * (long long)F1 * P2;
        for (int idx = tid; idx < TX * F1; idx += kThreads) {
            const int x = idx % TX, f1 = idx / TX;
            if (x >= width) continue;
            const float2 z1 = buf[x * LS + phys(f1)];
            const float2 z2 = buf[x * LS + phys((P1 - f1) & (P1 - 1))];
            float2 A0 = make_float2(0.5f * (z1.x + z2.x), 0.5f * (z1.y - z2.y));
            float2 A1 = make_float2(0.5f * (z1.y + z2.y), 0.5f * (z2.x - z1.x));
            const unsigned t2 = 2u * (c0 + x);
            A0 = cmul(A0, twiddle_p(p.twp, t2 * (unsigned)f1));
            A1 = cmul(A1, twiddle_p(p.twp, (t2 + 1u) * (unsigned)f1));
            HN_G(dst + (long long)f1 * P2 + t2, 16);
            *reinterpret_cast<float4 *>(dst + (long long)f1 * P2 + t2) = make_float4(A0.x, A0.y, A1.x, A1.y);
        }
        __syncthreads();
    }
}

struct CoreArgs {
    float2 *u;              // [slices][F1][P2], in place
    const float2 *h;        // [h slices][F1][P2]
    long long slices;
    int f1n;                // P1/2 + 1
    long long h_mod, h_off; // h slice = h_mod ? (s + h_off) % h_mod : s
    float scale;
    const float2 *tw2; int tw2_n;
    TwoLevel twp;
};

template <int LOG2P2>
__global__ void __launch_bounds__(kThreads) ct_core_kernel(CoreArgs p)
{
    constexpr int P2 = 1 << LOG2P2;
    constexpr int LS = line_stride(P2);
    extern __shared__ float2 smem[];
    const int G = tile_lines(LOG2P2);
    float2 *bu = smem;
    float2 *bh = smem + G * LS;
    float2 *tw = smem + 2 * G * LS;
    const int tid = threadIdx.x;
    load_twiddles(tw, p.tw2, P2, p.tw2_n, tid, kThreads);
    const long long rows = p.slices * p.f1n;
    const long long chunks = (rows + G - 1) / G;
    for (long long ch = blockIdx.x; ch < chunks; ch += gridDim.x) {
        for (int idx = tid; idx < G * P2; idx += kThreads) {
            const int g = idx / P2, t2 = idx % P2;
            const long long r = ch * G + g;
            float2 a = make_float2(0.f, 0.f), b = a;
            if (r < rows) {
                const long long s = r / p.f1n;
                const int f1 = (int)(r % p.f1n);
                const long long hs = p.h_mod ? (s + p.h_off) % p.h_mod : s;
                HN_G(p.u + r * P2 + t2, 8);
                HN_G(p.h + (hs * p.f1n + f1) * P2 + t2, 8);
                a = p.u[r * P2 + t2];
                b = __ldg(p.h + (hs * p.f1n + f1) * P2 + t2);
            }
            bu[g * LS + phys(t2)] = a;
            bh[g * LS + phys(t2)] = b;
        }
        __syncthreads();
        fft_lines<LOG2P2, false, PRUNE_NONE, kThreads>(bu, G, LS, tw, tid);
        fft_lines<LOG2P2, false, PRUNE_NONE, kThreads>(bh, G, LS, tw, tid);
        for (int idx = tid; idx < G * P2; idx += kThreads) {
            const int g = idx / P2, f2 = idx % P2;
            const int a = g * LS + phys(f2);
            const float2 w = cmul(bu[a], bh[a]);
            bu[a] = make_float2(w.x * p.scale, w.y * p.scale);
        }
        __syncthreads();
        fft_lines<LOG2P2, true, PRUNE_NONE, kThreads>(bu, G, LS, tw, tid);
        for (int idx = tid; idx < G * P2; idx += kThreads) {
            const int g = idx / P2, t2 = idx % P2;
            const long long r = ch * G + g;
            if (r >= rows) continue;
            const int f1 = (int)(r % p.f1n);
            const float2 w = twiddle_p(p.twp, (unsigned)t2 * (unsigned)f1);
            HN_G(p.u + r * P2 + t2, 8);
            p.u[r * P2 + t2] = cmulc(bu[g * LS + phys(t2)], w);
        }
        __syncthreads();
    }
}

struct ColsInvArgs {
    const float2 *in;       // [slices][F1][P2]
    const void *q;
    void *y;
    long long slices;
    int len;                // L
    int log2p2;
    const float2 *tw1; int tw1_n;
};

template <typename T, int LOG2P1>
__global__ void __launch_bounds__(kThreads) ct_cols_inv_kernel(ColsInvArgs p)
{
    constexpr int P1 = 1 << LOG2P1;
    constexpr int LS = line_stride(P1);
    constexpr int F1 = P1 / 2 + 1;
    extern __shared__ float2 smem[];
    const int TX = tile_lines(LOG2P1);
    float2 *buf = smem;
    float2 *tw = smem + TX * LS;
    const int tid = threadIdx.x;
    const T *pq = (const T *)p.q;
    T *py = (T *)p.y;
    load_twiddles(tw, p.tw1, P1, p.tw1_n, tid, kThreads);
    const int P2 = 1 << p.log2p2;
    const int tpc = (P2 / 2 + TX - 1) / TX;
    const long long tiles = p.slices * tpc;
    for (long long t = blockIdx.x; t < tiles; t += gridDim.x) {
        const long long s = t / tpc;
        const int c0 = (int)(t % tpc) * TX;
        const int width = P2 / 2 - c0 < TX ? P2 / 2 - c0 : TX;
        const float2 *src = p.in + s * (long long)F1 * P2;
        for (int idx = tid; idx < TX * P1; idx += kThreads) {
            const int x = idx % TX, pos = idx / TX;
            float2 c = make_float2(0.f, 0.f);
            if (x < width) {
                const bool mirror = pos > P1 / 2;
                const int f1 = mirror ? P1 - pos : pos;
                HN_G(src + (long long)f1 * P2 + 2 * (c0 + x), 16);
                float4 ab = *reinterpret_cast<const float4 *>(src + (long long)f1 * P2 + 2 * (c0 + x));
                if (mirror) { ab.y = -ab.y; ab.w = -ab.w; }
                c = make_float2(ab.x - ab.w, ab.y + ab.z);
            }
            buf[x * LS + phys(pos)] = c;
        }
        __syncthreads();
        fft_lines<LOG2P1, true, PRUNE_OUT, kThreads>(buf, TX, LS, tw, tid);
        const long long base = s * (long long)p.len;
        for (int idx = tid; idx < TX * (P1 / 2); idx += kThreads) {
            const int x = idx % TX, t1 = idx / TX;
            if (x >= width) continue;
            const long long tt = (long long)t1 * P2 + 2 * (c0 + x);
            const float2 z = buf[x * LS + phys(t1)];
            if (tt < p.len) IO<T>::st(py, base + tt, z.x * IO<T>::ld(pq, base + tt));
            if (tt + 1 < p.len) IO<T>::st(py, base + tt + 1, z.y * IO<T>::ld(pq, base + tt + 1));
        }
        __syncthreads();
    }
}

// ---- host side -----------------------------------------------------------------------------

static size_t smem_for(int log2n, int lines, int buffers)
{
    const int n = 1 << log2n;
    return sizeof(float2) * ((size_t)buffers * lines * line_stride(n) + n / 2);
}

#define HN_SWITCH_CT(x, CALL)                                                                   \
    switch (x) {                                                                                \
    case 7: CALL(7); break; case 8: CALL(8); break; case 9: CALL(9); break;                     \
    case 10: CALL(10); break; case 11: CALL(11); break; case 12: CALL(12); break;               \
    case 13: CALL(13); break;                                                                   \
    default: return -1;                                                                         \
    }

template <typename T, int LOG2P1>
static int launch_cols_fwd_t(const ColsFwdArgs &a, bool prune, cudaStream_t st)
{
    const int TX = tile_lines(LOG2P1);
    const size_t sm = smem_for(LOG2P1, TX, 1);
    const int P2 = 1 << a.log2p2;
    const long long tiles = a.slices * ((P2 / 2 + TX - 1) / TX);
    const int grid = (int)(tiles < (long long)sms() * 8 ? tiles : (long long)sms() * 8);
#define HN_LAUNCH(HASB, PR)                                                                     \
    do {                                                                                        \
        static DevOnce attr;                                                               \
        if (attr.first()) {                                                                            \
            cudaFuncSetAttribute(ct_cols_fwd_kernel<T, LOG2P1, HASB, PR>,                       \
                                 cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);         \
        }                                                                                       \
        ct_cols_fwd_kernel<T, LOG2P1, HASB, PR><<<grid, kThreads, sm, st>>>(a);                 \
    } while (0)
    if (a.b) HN_LAUNCH(true, true);
    else if (prune) HN_LAUNCH(false, true);
    else HN_LAUNCH(false, false);
#undef HN_LAUNCH
    return 1;
}

static int launch_cols_fwd(const ColsFwdArgs &a, int log2p1, bool prune, int dtype, cudaStream_t st)
{
    int n = 0;
#define CALLF(L) n = launch_cols_fwd_t<float, L>(a, prune, st)
#define CALLB(L) n = launch_cols_fwd_t<bf16, L>(a, prune, st)
    if (dtype == 0) { HN_SWITCH_CT(log2p1, CALLF) } else { HN_SWITCH_CT(log2p1, CALLB) }
#undef CALLF
#undef CALLB
    return n;
}

template <int LOG2P2> static int launch_core_t(const CoreArgs &a, cudaStream_t st)
{
    const int G = tile_lines(LOG2P2);
    const size_t sm = smem_for(LOG2P2, G, 2);
    const long long chunks = (a.slices * a.f1n + G - 1) / G;
    const int grid = (int)(chunks < (long long)sms() * 8 ? chunks : (long long)sms() * 8);
    static DevOnce attr;
    if (attr.first()) {
        cudaFuncSetAttribute(ct_core_kernel<LOG2P2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
    }
    ct_core_kernel<LOG2P2><<<grid, kThreads, sm, st>>>(a);
    return 1;
}

static int launch_core(const CoreArgs &a, int log2p2, cudaStream_t st)
{
    int n = 0;
#define CALLC(L) n = launch_core_t<L>(a, st)
    HN_SWITCH_CT(log2p2, CALLC)
#undef CALLC
    return n;
}

template <typename T, int LOG2P1> static int launch_cols_inv_t(const ColsInvArgs &a, cudaStream_t st)
{
    const int TX = tile_lines(LOG2P1);
    const size_t sm = smem_for(LOG2P1, TX, 1);
    const int P2 = 1 << a.log2p2;
    const long long tiles = a.slices * ((P2 / 2 + TX - 1) / TX);
    const int grid = (int)(tiles < (long long)sms() * 8 ? tiles : (long long)sms() * 8);
    static DevOnce attr;
    if (attr.first()) {
        cudaFuncSetAttribute(ct_cols_inv_kernel<T, LOG2P1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
    }
    ct_cols_inv_kernel<T, LOG2P1><<<grid, kThreads, sm, st>>>(a);
    return 1;
}

static int launch_cols_inv(const ColsInvArgs &a, int log2p1, int dtype, cudaStream_t st)
{
    int n = 0;
#define CALLF(L) n = launch_cols_inv_t<float, L>(a, st)
#define CALLB(L) n = launch_cols_inv_t<bf16, L>(a, st)
    if (dtype == 0) { HN_SWITCH_CT(log2p1, CALLF) } else { HN_SWITCH_CT(log2p1, CALLB) }
#undef CALLF
#undef CALLB
    return n;
}

static float2 *upload_table(GuardedAllocs *g, int n, double denom, double mult, size_t *bytes)
{
    std::vector<float2> t(n);
    for (int i = 0; i < n; ++i) {
        const double ang = -2.0 * M_PI * ((double)i * mult) / denom;
        t[i] = make_float2((float)cos(ang), (float)sin(ang));
    }
    float2 *d = nullptr;
    if (guarded_alloc(g, (void **)&d, sizeof(float2) * n) != cudaSuccess) { cudaGetLastError(); return nullptr; }
    if (cudaMemcpy(d, t.data(), sizeof(float2) * n, cudaMemcpyHostToDevice) != cudaSuccess) {
        cudaGetLastError(); return nullptr;          // the allocation stays on the plan's list and is freed with it
    }
    *bytes += sizeof(float2) * n;
    return d;
}

int ct1d_init(Ct1dPlan *c, int L, int K, int log2p, int B, int C, int causal, int dtype, const Switches &sw,
              GuardedAllocs *g, size_t *bytes)
{
    c->sw = sw;
    c->keep_filter = 0;
    c->dt_in = c->dt_out = c->dt_h = dtype;
    c->L = L; c->K = K; c->log2p = log2p; c->B = B; c->C = C; c->causal = causal; c->dtype = dtype;
    c->log2p1 = log2p / 2;
    c->log2p2 = log2p - c->log2p1;
    const int P1 = 1 << c->log2p1, P2 = 1 << c->log2p2;
    const long long per_slice = (long long)(P1 / 2 + 1) * P2;
    const long long S = (long long)B * C;
    long long spc = ((3ll << 30) / (long long)sizeof(float2)) / (2 * per_slice);
    if (spc < 1) spc = 1;
    if (spc > S) spc = S;
    c->slices_per_chunk = spc;
    c->wh_slices = spc > C ? spc : C;
    *bytes = 0;
    c->lo = log2p / 2;
    c->tw1 = upload_table(g, P1, (double)P1, 1.0, bytes);
    c->tw2 = upload_table(g, P2, (double)P2, 1.0, bytes);
    c->twp_fine = upload_table(g, 1 << c->lo, ldexp(1.0, log2p), 1.0, bytes);
    c->twp_coarse = upload_table(g, 1 << (log2p - c->lo), ldexp(1.0, log2p), ldexp(1.0, c->lo), bytes);
    if (!c->tw1 || !c->tw2 || !c->twp_fine || !c->twp_coarse) return 3;
    size_t need = sizeof(float2) * per_slice * spc;
    if (guarded_alloc(g, (void **)&c->wu, need) != cudaSuccess) { cudaGetLastError(); *bytes = need; return 3; }
    *bytes += need;
    need = sizeof(float2) * per_slice * c->wh_slices;
    if (guarded_alloc(g, (void **)&c->wh, need) != cudaSuccess) { cudaGetLastError(); *bytes = need; return 3; }
    *bytes += need;
    return 0;
}

static int filter_pass(Ct1dPlan *c, const char *h, long long n, cudaStream_t st, int *launches, Prof *prof)
{
    ColsFwdArgs a{};
    a.a = h; a.b = nullptr; a.out = c->wh; a.slices = n; a.in_slice = c->K; a.len = c->K;
    a.shift = c->causal ? 0 : c->L - 1;
    a.log2p2 = c->log2p2; a.tw1 = c->tw1; a.tw1_n = 1 << c->log2p1;
    a.twp = TwoLevel{c->twp_coarse, c->twp_fine, c->lo};
    prof->begin(KID_CT_COLS_H, st);
    int r = launch_cols_fwd(a, c->log2p1, c->causal != 0, c->dt_h, st);
    prof->end(st);
    if (r < 0) return -1;
    *launches += r;
    return 0;
}

int ct1d_forward(Ct1dPlan *c, const void *q, const void *k, const void *v, const void *h, bool shared,
                 void *y, cudaStream_t st, int *launches, Prof *prof)
{
    const size_t ei = c->dt_in == 0 ? 4 : 2, eo = c->dt_out == 0 ? 4 : 2, eh = c->dt_h == 0 ? 4 : 2;
    const TwoLevel twp{c->twp_coarse, c->twp_fine, c->lo};
    if (ct1d_uses_w(c)) {
        const bool staged_ok = c->causal != 0;
        if (shared && c->r0 == 0 && !c->keep_filter && ct1d_w_filter(c, h, c->C, staged_ok, st, launches, prof, filter_pass)) return -1;
        for (long long s0 = c->r0; s0 < c->r1; s0 += c->slices_per_chunk) {
            const long long n = c->r1 - s0 < c->slices_per_chunk ? c->r1 - s0 : c->slices_per_chunk;
            if (!shared && ct1d_w_filter(c, (const char *)h + (size_t)s0 * c->K * eh, n, staged_ok, st, launches, prof, filter_pass))
                return -1;
            if (ct1d_w_body(c, (const char *)q + (size_t)s0 * c->L * eo, (const char *)k + (size_t)s0 * c->L * ei,
                            (const char *)v + (size_t)s0 * c->L * ei, n, shared, s0, (char *)y + (size_t)s0 * c->L * eo,
                            st, launches, prof))
                return -1;
        }
        return 0;
    }
    if (shared && c->r0 == 0 && !c->keep_filter && filter_pass(c, (const char *)h, c->C, st, launches, prof)) return -1;
    for (long long s0 = c->r0; s0 < c->r1; s0 += c->slices_per_chunk) {
        const long long n = c->r1 - s0 < c->slices_per_chunk ? c->r1 - s0 : c->slices_per_chunk;
        if (!shared && filter_pass(c, (const char *)h + (size_t)s0 * c->K * eh, n, st, launches, prof)) return -1;
        ColsFwdArgs a{};
        a.a = (const char *)k + (size_t)s0 * c->L * ei; a.b = (const char *)v + (size_t)s0 * c->L * ei;
        a.out = c->wu; a.slices = n; a.in_slice = c->L; a.len = c->L; a.shift = 0;
        a.log2p2 = c->log2p2; a.tw1 = c->tw1; a.tw1_n = 1 << c->log2p1; a.twp = twp;
        prof->begin(KID_CT_COLS_U, st);
        int r = launch_cols_fwd(a, c->log2p1, true, c->dt_in, st);
        prof->end(st);
        if (r < 0) return -1;
        *launches += r;
        CoreArgs cr{};
        cr.u = c->wu; cr.h = c->wh; cr.slices = n; cr.f1n = (1 << c->log2p1) / 2 + 1;
        cr.h_mod = shared ? c->C : 0; cr.h_off = shared ? s0 % c->C : 0;
        cr.scale = (float)ldexp(1.0, -c->log2p);
        cr.tw2 = c->tw2; cr.tw2_n = 1 << c->log2p2; cr.twp = twp;
        prof->begin(KID_CT_CORE, st);
        r = launch_core(cr, c->log2p2, st);
        prof->end(st);
        if (r < 0) return -1;
        *launches += r;
        ColsInvArgs ci{};
        ci.in = c->wu; ci.q = (const char *)q + (size_t)s0 * c->L * eo; ci.y = (char *)y + (size_t)s0 * c->L * eo;
        ci.slices = n; ci.len = c->L; ci.log2p2 = c->log2p2; ci.tw1 = c->tw1; ci.tw1_n = 1 << c->log2p1;
        prof->begin(KID_CT_COLS_INV, st);
        r = launch_cols_inv(ci, c->log2p1, c->dt_out, st);
        prof->end(st);
        if (r < 0) return -1;
        *launches += r;
    }
    return 0;
}

// the warp-engine kernels serve a forward when they take every element type it uses
bool ct1d_uses_w(const Ct1dPlan *c)
{
    if (c->sw.force_generic) return false;
    const int dts[4] = {c->dtype, c->dt_in, c->dt_out, c->dt_h};
    for (int i = 0; i < 4; ++i)
        if (!ct1d_w_supported(c->log2p1, c->log2p2, c->L, c->K, c->causal, dts[i])) return false;
    return true;
}

// The warp-engine kernels need 16-byte rows in the given type; the block-wide kernels take either type as it is.  A plan
// must not change kernel family between forwards (the filter workspace layouts differ), so a type is accepted when it
// leaves the family the plan's own type selects.
bool ct1d_takes_dtype(const Ct1dPlan *c, int dtype)
{
    if (dtype == c->dtype) return true;
    const bool w_own = !c->sw.force_generic && ct1d_w_supported(c->log2p1, c->log2p2, c->L, c->K, c->causal, c->dtype);
    if (!w_own) return true;
    return ct1d_w_supported(c->log2p1, c->log2p2, c->L, c->K, c->causal, dtype);
}

int ct1d_launches(const Ct1dPlan *c, bool shared)
{
    const long long S = (long long)c->B * c->C;
    const long long chunks = (S + c->slices_per_chunk - 1) / c->slices_per_chunk;
    if (ct1d_uses_w(c)) return (int)(shared ? 2 + 3 * chunks : 5 * chunks);
    return (int)(shared ? 1 + 3 * chunks : 4 * chunks);
}

}  // namespace hn
