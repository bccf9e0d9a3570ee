// Plane-fused kernels for 3-D grids (and the building blocks of the fused 2-D path).
//
// One CTA transforms a whole x-y plane on chip, so the two in-plane axes cost
// one trip through HBM instead of two (the paper's nSubQ keeps intermediates in
// shared memory the same way for 1-D and 2-D; it describes no 3-D kernel):
//
//   uplane     k*v plane: gate, zero-pad, real-to-complex along x (two real rows
//              per complex transform, separated by the column transform as it loads),
//              transpose through a shared-memory column store, complex transform
//              along y.  Output lines are [kx][ky], at twice their value.
//   hplane     filter plane, which has twice the rows and columns: the even and the odd
//              bins along x are produced one after the other (one radix-2
//              decimation-in-frequency step applied to the taps as they are read), each
//              half filling a column store of the size of a k*v plane's.  The tap rows are
//              fetched once: the odd half's inputs wait in tensor memory meanwhile.
//              Output at twice its value as well (the core's scale carries both factors).
//   plane_inv  inverse along y (keeping the cropped rows; two rows combined into one
//              complex row as they leave the registers), inverse complex-to-real
//              along x, crop, output gate q, store.
//
// The stores hold the RAW transforms of the row pairs, [bin][row pair]; a column reads its bin and the mirrored one.
// The two purely real bins of every row (kx = 0 and kx = P/2) travel as one complex column, so a plane has
// exactly P/2 columns.
#include "common.cuh"
#include "planes.cuh"
#include "wfft.cuh"
#include "plane_util.cuh"
#include "tmem_util.cuh"

namespace hn {

template <int LOG2P> struct PlaneCfg {
    static constexpr int P = 1 << LOG2P, HP = P / 2, XH = HP + 1;
    static constexpr int CSS = HP + 1;                       // filter planes: store stride (odd), P/2 bins of P/2 row pairs per half
    using F = WF<LOG2P, false>;
    using FI = WF<LOG2P, true>;
    using FH = WF<LOG2P - 1, false>;                         // half-length rows of hplane
    static constexpr int NG = kPlaneThreads / F::TPL;        // groups working on P-point lines
    static constexpr int NGH = kPlaneThreads / FH::TPL;      // groups working on P/2-point lines
    static constexpr int LS = plane_ls(P);
    static constexpr int LSH = plane_ls(HP);
    static constexpr int WBUF = (NG * LS > NGH * LSH) ? NG * LS : NGH * LSH;
    static constexpr int CSU = P / 4 + 1;                    // k*v planes: P bins of P/4 row pairs (odd stride)
    static constexpr int CSN = (HP * CSS > P * CSU) ? HP * CSS : P * CSU;       // column store, entries
    static constexpr size_t TMP = (size_t)CSN + WBUF + P + HP + 2 * P;          // P entries: raw transform of the packed column
    static constexpr size_t SMEM = sizeof(float2) * (TMP + P + 2);      // + the slot that receives the tensor-memory base
};

template <int LOG2P> __device__ __forceinline__ void load_plane_twiddles(float2 *tw, float2 *twh, const float2 *gtw, int gtw_n, int tid)
{
    constexpr int P = 1 << LOG2P;
    const int step = gtw_n >> LOG2P;
    for (int t = tid; t < P; t += kPlaneThreads) { HN_G(gtw + t * step, 8); tw[t] = gtw[t * step]; }
    for (int t = tid; t < P / 2; t += kPlaneThreads) { HN_G(gtw + 2 * t * step, 8); twh[t] = gtw[2 * t * step]; }
}

// ---- k*v planes ---------------------------------------------------------------------------------

template <typename T, int LOG2P>
__global__ void __launch_bounds__(kPlaneThreads, 1) uplane_kernel(PlaneArgs p)
{
    using C = PlaneCfg<LOG2P>;
    using F = typename C::F;
    using PC0 = typename F::template Pass<0>;
    constexpr int P = C::P, HP = C::HP, QP = P / 4, TPL = F::TPL, CSU = C::CSU;
    constexpr unsigned FULL = 0xffffffffu;                   // every warp runs the loops below in step: whole-warp barriers
    static_assert(QP % C::NG == 0 || C::NG % QP == 0, "whole warps take part in the row loop");
    static_assert(HP % C::NG == 0 || C::NG % HP == 0, "whole warps take part in the column loop");
    extern __shared__ float2 smem[];
    float2 *cs = smem;
    float2 *wbuf = cs + C::CSN;
    float2 *tw = wbuf + C::WBUF;
    float2 *twh = tw + P;
    float2 *tmp = smem + C::TMP;
    const int tid = threadIdx.x, l = tid % TPL, gid = tid / TPL;
    float2 *line = wbuf + gid * C::LS;
    load_plane_twiddles<LOG2P>(tw, twh, p.gtw, p.gtw_n, tid);
    __syncthreads();
    PlaneTw<LOG2P, false> twp;
    twp.init(l, tw, twh + HP, tid, kPlaneThreads);
    __syncthreads();
    const T *pk = (const T *)p.a;
    const T *pv = (const T *)p.b;
    const unsigned char *kb = (const unsigned char *)p.a, *vb = (const unsigned char *)p.b;
    const unsigned char *ke = kb + p.a_elems * sizeof(T), *ve = vb + p.a_elems * sizeof(T);
    const int Lx = p.lx, Ly = p.ly;
    for (long long pl = blockIdx.x; pl < p.planes; pl += gridDim.x) {
        const long long ib = pl * (long long)Ly * Lx;
        // rows: y and y + P/4 share a transform (rows P/4 .. Ly-1 exist, Ly > P/4; a missing partner is a zero row)
        for (int rp = gid; rp < QP; rp += C::NG) {
            const int y1 = rp + QP;
            const bool has1 = y1 < Ly;
            // the rows of k and of v are fetched with 16-byte copies into the line itself, which the first pass reads
            // before anything is written to it
            constexpr int SLOT = HP * (int)sizeof(T) + 32;
            static_assert(4 * SLOT <= C::LS * 8, "staged rows must fit the line");
            unsigned char *sk0 = reinterpret_cast<unsigned char *>(line), *sk1 = sk0 + SLOT, *sv0 = sk1 + SLOT, *sv1 = sv0 + SLOT;
            const int rowb = Lx * (int)sizeof(T);
            const unsigned char *gk0 = kb + (ib + (long long)rp * Lx) * sizeof(T), *gk1 = gk0 + (long long)QP * rowb;
            const unsigned char *gv0 = vb + (ib + (long long)rp * Lx) * sizeof(T), *gv1 = gv0 + (long long)QP * rowb;
            stage_row_u<TPL, HP * (int)sizeof(T)>(sk0, gk0, rowb, kb, ke, l);
            stage_row_u<TPL, HP * (int)sizeof(T)>(sv0, gv0, rowb, vb, ve, l);
            if (has1) {
                stage_row_u<TPL, HP * (int)sizeof(T)>(sk1, gk1, rowb, kb, ke, l);
                stage_row_u<TPL, HP * (int)sizeof(T)>(sv1, gv1, rowb, vb, ve, l);
            }
            cp_async_wait_all();
            __syncwarp();
            const T *k0 = reinterpret_cast<const T *>(sk0 + ((unsigned long long)gk0 & 15ull)) + l;
            const T *v0 = reinterpret_cast<const T *>(sv0 + ((unsigned long long)gv0 & 15ull)) + l;
            const T *k1 = reinterpret_cast<const T *>(sk1 + ((unsigned long long)gk1 & 15ull)) + l;
            const T *v1 = reinterpret_cast<const T *>(sv1 + ((unsigned long long)gv1 & 15ull)) + l;
            float2 z0 = make_float2(0.f, 0.f), zh = z0;
            // The raw transform Z of the row pair goes straight into the store [bin][row pair]; the column transform
            // separates the two rows as it loads.
            auto keep = [&](int, int r, int kk, float2 z) {
                cs[kk * CSU + rp] = z;
                if (r == 0) z0 = z;                           // lane 0: bins 0 and P/2
                if (r == F::LastPass::R / 2) zh = z;
            };
            if (Lx == HP && has1) {
                // full rows: no bounds tests in the input functor
                F::template run<PRUNE_IN, true>(l, FULL, twp, line, [&](int i, int r, int) {
                    const int x = i * TPL + r * (P / PC0::R);                   // + l
                    return make_float2((float)k0[x] * (float)v0[x], (float)k1[x] * (float)v1[x]);
                }, keep);
            } else {
                F::template run<PRUNE_IN, true>(l, FULL, twp, line, [&](int i, int r, int idx) {
                    const int x = i * TPL + r * (P / PC0::R);
                    float a = 0.f, b = 0.f;
                    if (idx < Lx) {
                        a = (float)k0[x] * (float)v0[x];
                        if (has1) b = (float)k1[x] * (float)v1[x];
                    }
                    return make_float2(a, b);
                }, keep);
            }
            if (l == 0) {
                // Bins 0 and P/2 (both held by lane 0) are the real bins of the two rows: Z[0] = (F_y[0], F_y'[0]),
                // Z[P/2] = (F_y[P/2], F_y'[P/2]).  They travel as one column (kx = 0, mirrored bin P/2): with
                // a = (Z0.x - Zh.y, Z0.y + Zh.x), b = (Z0.x + Zh.y, Z0.y - Zh.x) the column phase's separation
                // gives a + conj b = 2 (Z0.x, Zh.x) and -i (a - conj b) = 2 (Z0.y, Zh.y).
                static_assert(F::LastPass::IPL == 1 && HP % (P / F::LastPass::R) == 0, "lane 0 holds bins 0 and P/2");
                cs[rp] = make_float2(z0.x - zh.y, z0.y + zh.x);
                cs[HP * CSU + rp] = make_float2(z0.x + zh.y, z0.y - zh.x);
            }
            __syncwarp();
        }
        __syncthreads();
        // columns: with Z the raw transform of row pair (y, y + P/4),
        //   2 F_y[kx] = Z[kx] + conj Z[P - kx],   2 F_{y+P/4}[kx] = -i (Z[kx] - conj Z[P - kx]);
        // a lane's first-pass inputs y = j + r P/R, r < R/2 (the rest is padding), come from the row pairs of r < R/4,
        // both members each.  Values leave at twice their size (the factor 1/2 is left to the spectral core's scale).
        float2 *dst = p.out + pl * (long long)C::XH * P;
        if (pl + gridDim.x < p.planes) {
            // the next plane's rows travel to L2 during the column phase, which loads nothing from global memory
            const long long nb = (pl + gridDim.x) * (long long)Ly * Lx;
            prefetch_l2(pk + nb, (long long)Ly * Lx * sizeof(T), tid);
            prefetch_l2(pv + nb, (long long)Ly * Lx * sizeof(T), tid);
        }
        for (int kx = gid; kx < HP; kx += C::NG) {
            // Column 0 packs bins kx = 0 and kx = P/2 of every row as one complex number; it runs the same transform as
            // every other column (the group that shares its warp does not wait for a second code path), its raw transform
            // goes to a shared-memory line and is unpacked after the column phase.
            const bool packed = kx == 0;
            const float2 *ca = cs + kx * CSU, *cb = cs + (packed ? HP : P - kx) * CSU;
            float2 *d = packed ? tmp : dst + (long long)kx * P;
            float2 second[PC0::IPL][PC0::R / 4] = {};
            F::template run<PRUNE_IN>(l, FULL, twp, line,
                [&](int i, int r, int idx) {
                    if (r >= PC0::R / 4) return second[i][r - PC0::R / 4];
                    const float2 za = ca[idx], zm = cb[idx];
                    second[i][r] = make_float2(za.y + zm.y, zm.x - za.x);
                    return make_float2(za.x + zm.x, za.y - zm.y);
                },
                [&](int, int, int idx, float2 v) { HN_G(d + idx, 8); d[idx] = v; });
            __syncwarp();
        }
        __syncthreads();
        if (tid < P) {
            // C = raw transform of the packed column: bins kx = 0 and kx = P/2 are (C[ky] + conj C[-ky]) / 2 and
            // -i (C[ky] - conj C[-ky]) / 2.  (The line is next written after the next CTA barrier.)
            const int ky = tid;
            const float2 c1 = tmp[ky], c2 = tmp[(P - ky) & (P - 1)];
            float2 *dn = dst + (long long)HP * P;
            HN_G(dst + ky, 8);
            HN_G(dn + ky, 8);
            dst[ky] = make_float2(0.5f * (c1.x + c2.x), 0.5f * (c1.y - c2.y));
            dn[ky] = make_float2(0.5f * (c1.y + c2.y), 0.5f * (c2.x - c1.x));
        }
    }
}

// ---- filter planes ----------------------------------------------------------------------------------

// A filter plane has P rows of P taps: twice the rows and columns of a k*v plane, too much for one
// column store.  The transform along x is split by one decimation-in-frequency step: the even bins
// of a row are the half-length transform of f[x] + f[x + P/2], the odd bins that of
// (f[x] - f[x + P/2]) W_P^x.  Each half (e = 0: even kx, e = 1: odd kx) fills a column store of
// P/4 columns by P rows, whose columns are then transformed along y and written out as whole lines.
//
// Two real rows share one complex row transform: padded rows y and y + P/2 (row pair p = y mod P/2).  They are NOT
// separated after it: the raw transform Z of every row pair goes straight from the last pass's registers into the
// store [bin k][row pair], and the column transform of bin k separates them as it loads.  A lane's first-pass inputs
// y = j + r P/R come from the row pairs p = j + r P/R, r < R/2, both members each, so one pair of loads (Z[k] and the
// mirrored bin Z[k']) yields two inputs:
//   2 F_y[k] = Z[k] + conj Z[k'],   2 F_{y+P/2}[k] = -i (Z[k] - conj Z[k']),
// k' = (H - k) mod H in the even half, H - 1 - k in the odd one (H = P/2 bins per half).  Separated values come out at
// twice their value (the factor 1/2 is left to the spectral core's scale).
//
// Tap rows are staged so that no index wraps: padded position x holds tap (x + Lx - 1) mod P, so the P positions of
// a row are a window W of P consecutive tap indices starting at -(P/2 + 1 - Lx), with zeros outside [0, Kx):
// position x + P/2 is W[x], position x is W[x + P/2] (x < P/2).  A thread's taps sit at constant offsets from one
// address.  The tap rows are fetched and unpacked once per plane: while a thread prepares the even half it also forms
// its inputs of the odd half, f[x] - f[x + P/2], and parks them in tensor memory (its own lane, 2 * points-per-thread
// columns per row pair); the odd half reads them back instead of staging the rows again.
//
// The purely real bins kx = 0 and kx = P/2 of every row travel as one complex column (column 0 of the even half): its
// store entries are rewritten by the row phase so that the common separation formulas deliver (2 F_y[0], 2 F_y[P/2])
// for it; its raw transform goes to a shared-memory line, which the whole CTA unpacks into lines 0 and P/2 of the
// output after the column phase.
template <typename T, int LOG2P>
__global__ void __launch_bounds__(kPlaneThreads, 1) hplane_kernel(PlaneArgs p)
{
    using C = PlaneCfg<LOG2P>;
    using F = typename C::F;
    using FH = typename C::FH;
    constexpr int P = C::P, HP = C::HP, QP = P / 4, TPL = F::TPL, TPLH = FH::TPL;
    constexpr int CS2 = HP + 1;                              // store stride (odd): HP bins of HP row pairs, raw row transforms
    static_assert(HP * CS2 <= HP * C::CSS, "store of a half fits the plane buffer");
    extern __shared__ float2 smem[];
    float2 *cs = smem;
    float2 *wbuf = cs + C::CSN;
    float2 *tw = wbuf + C::WBUF;
    float2 *twh = tw + P;
    float2 *tmp = smem + C::TMP;
    const int tid = threadIdx.x;
    const int l = tid % TPL, gid = tid / TPL;
    const int lh = tid % TPLH, gidh = tid / TPLH;
    constexpr unsigned FULL = 0xffffffffu;                   // every warp runs the loops below in step: whole-warp barriers
    float2 *line = wbuf + gid * C::LS;
    float2 *lineh = wbuf + gidh * C::LSH;
    using PH0 = typename FH::template Pass<0>;
    using PC0 = typename F::template Pass<0>;
    constexpr int NPT = 2 * PH0::IPL * PH0::R;               // parked values per thread and row pair
    constexpr int ROUNDS = HP / C::NGH;                      // row pairs per lane group and half
    constexpr int TCOLS = 4 * ROUNDS * NPT;                  // four warps share each 32-lane quadrant
    static_assert(HP % C::NGH == 0 && TCOLS >= 32 && TCOLS <= 512 && (TCOLS & (TCOLS - 1)) == 0, "tensor-memory columns");
    static_assert(QP % C::NG == 0 || C::NG % QP == 0, "whole warps take part in the column loop");
    const int warp = tid >> 5;
    unsigned *tslot = reinterpret_cast<unsigned *>(smem + C::TMP + P);
    if (warp == 0) tmem_alloc((unsigned)__cvta_generic_to_shared(tslot), TCOLS);
    load_plane_twiddles<LOG2P>(tw, twh, p.gtw, p.gtw_n, tid);
    tmem_fence_before_sync();
    __syncthreads();
    tmem_fence_after_sync();
    const unsigned tbase = *tslot;
    const unsigned tpark = tmem_addr(tbase, warp, (warp >> 2) * ROUNDS * NPT);
    PlaneTw<LOG2P, false> twp;
    twp.init(l, tw, twh + HP, tid, kPlaneThreads);
    PassTw<LOG2P - 1, false> twr;                            // half-length rows
    twr.base = twh + HP + P;
    PassTw<LOG2P - 1, false>::build(twh + HP + P, p.gtw, p.gtw_n, tid, kPlaneThreads);
    __syncthreads();
    const unsigned char *hb = (const unsigned char *)p.a;
    const int Lx = p.lx, Ly = p.ly, Kx = 2 * Lx - 1, Ky = 2 * Ly - 1;
    constexpr int R0 = PH0::R;
    const int J0 = HP + 1 - Lx;                              // window position of tap 0
    const int RU = (J0 * (int)sizeof(T) + 15) & ~15;         // bytes kept free before the first copied chunk
    for (long long pl = blockIdx.x; pl < p.planes; pl += gridDim.x) {
        const long long ib = pl * (long long)Ky * Kx;
        float2 *dst = p.out + pl * (long long)C::XH * P;
        for (int e = 0; e < 2; ++e) {
            // the next plane's taps travel to L2 during the second half, when this plane's are on chip
            if (e == 1 && pl + gridDim.x < p.planes)
                prefetch_l2(hb + (pl + gridDim.x) * (long long)Ky * Kx * sizeof(T), (long long)Ky * Kx * sizeof(T), tid);
            if (e == 1 && tid < P) {
                // the raw transform C of the packed column (bins kx = 0 and kx = P/2 of every row) waits in a shared-memory
                // line since the column phase that has just ended: the two bins are (C[ky] + conj C[-ky]) / 2 and
                // -i (C[ky] - conj C[-ky]) / 2.  (The line is next written two CTA barriers from here.)
                const int ky = tid;
                const float2 c1 = tmp[ky], c2 = tmp[(P - ky) & (P - 1)];
                float2 *dn = dst + (long long)HP * P;
                HN_G(dst + ky, 8);
                HN_G(dn + ky, 8);
                dst[ky] = make_float2(0.5f * (c1.x + c2.x), 0.5f * (c1.y - c2.y));
                dn[ky] = make_float2(0.5f * (c1.y + c2.y), 0.5f * (c2.x - c1.x));
            }
            // rows: padded row y holds tap row (y + Ly - 1) mod P; rows y and y + P/2 share a transform (at most one
            // of the two lies in the zero band, which is shorter than P/2 rows)
            int round = 0;
            // the two groups of a half warp take row pairs 8 apart, so their stores (one row pair per group, consecutive
            // bins per lane) fall into different banks
            for (int rp = spread_pair<8>(gidh); rp < HP; rp += C::NGH, ++round) {
                const int my0 = (rp + Ly - 1) & (P - 1), my1 = my0 ^ HP;
                const bool v0 = my0 < Ky, v1 = my1 < Ky;
                // STAGED: both tap rows are fetched with 16-byte copies into the line itself, which
                // the first pass reads before anything is written to it; 4-byte taps do not fit the
                // half-length line and are read from global memory (L2) directly
                constexpr bool STAGED = sizeof(T) == 2;
                constexpr int SLOT = 4 * HP + 48;            // bytes kept per staged row: window, alignment slack, last chunk
                static_assert(!STAGED || 2 * SLOT + 32 <= C::LSH * 8, "staged rows must fit the line");
                // the four lines of a warp start 0, 64, 0, 64 bytes into the 128-byte bank row:
                // lines 2 and 3 stage 32 bytes further in, so the narrow tap loads do not collide
                unsigned char *s0 = reinterpret_cast<unsigned char *>(lineh) + 16 * (gidh & 2), *s1 = s0 + SLOT;
                const unsigned char *g0 = hb + (ib + (long long)my0 * Kx) * sizeof(T);
                const unsigned char *g1 = hb + (ib + (long long)my1 * Kx) * sizeof(T);
                const int n0 = v0 ? Kx : 0, n1 = v1 ? Kx : 0;
                float dd[NPT];                                // this thread's inputs of the odd half, before the twiddle
                float ss[NPT];                                // and of the even half
                const unsigned tcol = tpark + round * NPT;
                if (e == 0) {
                    if constexpr (STAGED) {
                        const int f0 = (int)((unsigned long long)g0 & 15ull), f1 = (int)((unsigned long long)g1 & 15ull);
                        if (v0) stage_row_u<TPLH, (2 * HP - 1) * (int)sizeof(T)>(s0 + RU, g0, Kx * (int)sizeof(T), hb, hb + p.a_elems * sizeof(T), lh);
                        if (v1) stage_row_u<TPLH, (2 * HP - 1) * (int)sizeof(T)>(s1 + RU, g1, Kx * (int)sizeof(T), hb, hb + p.a_elems * sizeof(T), lh);
                        cp_async_wait_all();
                        __syncwarp();
                        // window element j sits at w + 2 j; blank what lies outside the row once, so the tap loads
                        // need no bounds test
                        unsigned char *w0 = s0 + RU + f0 - J0 * (int)sizeof(T), *w1 = s1 + RU + f1 - J0 * (int)sizeof(T);
                        for (int j = lh; j < J0; j += TPLH) {
                            *reinterpret_cast<T *>(w0 + j * sizeof(T)) = T(0.f);
                            *reinterpret_cast<T *>(w1 + j * sizeof(T)) = T(0.f);
                        }
                        for (int j = J0 + n0 + lh; j < P; j += TPLH) *reinterpret_cast<T *>(w0 + j * sizeof(T)) = T(0.f);
                        for (int j = J0 + n1 + lh; j < P; j += TPLH) *reinterpret_cast<T *>(w1 + j * sizeof(T)) = T(0.f);
                        __syncwarp();
                        const T *t0 = reinterpret_cast<const T *>(w0) + lh, *t1 = reinterpret_cast<const T *>(w1) + lh;
#pragma unroll
                        for (int i = 0; i < PH0::IPL; ++i)
#pragma unroll
                            for (int r = 0; r < R0; ++r) {
                                const int x = i * TPLH + r * (HP / R0);          // + lh: position of this input
                                const float a0 = (float)t0[x + HP], b0 = (float)t0[x], a1 = (float)t1[x + HP], b1 = (float)t1[x];
                                ss[2 * (i * R0 + r)] = a0 + b0;
                                ss[2 * (i * R0 + r) + 1] = a1 + b1;
                                dd[2 * (i * R0 + r)] = a0 - b0;
                                dd[2 * (i * R0 + r) + 1] = a1 - b1;
                            }
                    } else {
                        const T *r0 = reinterpret_cast<const T *>(g0), *r1 = reinterpret_cast<const T *>(g1);
#pragma unroll
                        for (int i = 0; i < PH0::IPL; ++i)
#pragma unroll
                            for (int r = 0; r < R0; ++r) {
                                const int x = lh + i * TPLH + r * (HP / R0);
                                const int ta = x + Lx - 1, tb = x - J0;          // tap indices of positions x and x + P/2
                                const float a0 = ta < n0 ? IO<T>::ld(r0, ta) : 0.f, a1 = ta < n1 ? IO<T>::ld(r1, ta) : 0.f;
                                const float b0 = (tb >= 0 && tb < n0) ? IO<T>::ld(r0, tb) : 0.f;
                                const float b1 = (tb >= 0 && tb < n1) ? IO<T>::ld(r1, tb) : 0.f;
                                ss[2 * (i * R0 + r)] = a0 + b0;
                                ss[2 * (i * R0 + r) + 1] = a1 + b1;
                                dd[2 * (i * R0 + r)] = a0 - b0;
                                dd[2 * (i * R0 + r) + 1] = a1 - b1;
                            }
                    }
                    __syncwarp();                             // the whole warp parks together; every lane has read its taps
                    TmemIO<NPT>::st(tcol, dd);
                    tmem_wait_st();
                    float2 z0 = make_float2(0.f, 0.f), zh = z0;
                    FH::template run<PRUNE_NONE, false>(lh, FULL, twr, lineh,
                        [&](int i, int r, int) { return make_float2(ss[2 * (i * R0 + r)], ss[2 * (i * R0 + r) + 1]); },
                        [&](int, int r, int kk, float2 z) {
                            cs[kk * CS2 + rp] = z;
                            if (r == 0) z0 = z;                                  // lane 0: bins 0 and H/2
                            if (r == FH::LastPass::R / 2) zh = z;
                        });
                    if (lh == 0) {
                        // Bins 0 and H/2 (both held by lane 0) are the real bins kx = 0 and kx = P/2 of the two rows:
                        // Z[0] = (F_y[0], F_y'[0]), Z[H/2] = (F_y[P/2], F_y'[P/2]).  They travel as one column (k = 0, mirrored
                        // bin H/2): with a = (Z0.x - Zh.y, Z0.y + Zh.x), b = (Z0.x + Zh.y, Z0.y - Zh.x) the column phase's
                        // separation gives a + conj b = 2 (Z0.x, Zh.x) and -i (a - conj b) = 2 (Z0.y, Zh.y).
                        static_assert(FH::LastPass::IPL == 1 && (HP / 2) % (HP / FH::LastPass::R) == 0, "lane 0 holds bins 0 and H/2");
                        cs[rp] = make_float2(z0.x - zh.y, z0.y + zh.x);
                        cs[(HP / 2) * CS2 + rp] = make_float2(z0.x + zh.y, z0.y - zh.x);
                    }
                } else {
                    __syncwarp();
                    TmemIO<NPT>::ld(dd, tcol);
                    tmem_wait_ld();
                    FH::template run<PRUNE_NONE, false>(lh, FULL, twr, lineh,
                        [&](int i, int r, int idx) { return cmul(make_float2(dd[2 * (i * R0 + r)], dd[2 * (i * R0 + r) + 1]), tw[idx]); },
                        [&](int, int, int kk, float2 z) { cs[kk * CS2 + rp] = z; });
                }
                __syncwarp();
            }
            __syncthreads();
            // columns: P-point transforms over y of the bins kx = 2k + e
            for (int k = gid; k < QP; k += C::NG) {
                const bool packed = e == 0 && k == 0;
                const int km = packed ? HP / 2 : (e == 0 ? ((HP - k) & (HP - 1)) : HP - 1 - k);
                const float2 *ca = cs + k * CS2, *cb = cs + km * CS2;
                float2 *d = packed ? tmp : dst + (long long)(2 * k + e) * P;
                float2 second[PC0::IPL][PC0::R / 2] = {};     // inputs y + P/2, formed with their partners y
                F::template run<PRUNE_NONE>(l, FULL, twp, line,
                    [&](int i, int r, int idx) {
                        if (r >= PC0::R / 2) return second[i][r - PC0::R / 2];
                        const float2 za = ca[idx], zm = cb[idx];
                        second[i][r] = make_float2(za.y + zm.y, zm.x - za.x);
                        return make_float2(za.x + zm.x, za.y - zm.y);
                    },
                    [&](int, int, int idx, float2 v) { HN_G(d + idx, 8); d[idx] = v; });
                __syncwarp();
            }
            __syncthreads();
        }
    }
    // every warp's last tensor-memory read was waited for before the barrier above; the allocating warp frees
    tmem_fence_before_sync();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tbase, TCOLS);
}


// ---- inverse planes ------------------------------------------------------------------------------------

// VST: rows are whole numbers of 16-byte vectors and q, y are 16-byte aligned: the cropped rows go through the line
// once more and leave as 16-byte stores (gate values arrive as 16-byte loads); else one element per lane and leg.
// TWO: a second gate and result of the same planes, y2 = q2 * planes (the backward pass: dk = v du, dv = k du)
template <typename T, int LOG2P, bool VST, bool TWO>
__global__ void __launch_bounds__(kPlaneThreads, 1) plane_inv_kernel(PlaneArgs p)
{
    using C = PlaneCfg<LOG2P>;
    using FI = typename C::FI;
    constexpr int P = C::P, HP = C::HP, QP = P / 4, TPL = FI::TPL, CSI = C::CSU;
    extern __shared__ float2 smem[];
    float2 *cs = smem;
    float2 *wbuf = cs + C::CSN;
    float2 *tw = wbuf + C::WBUF;
    float2 *twh = tw + P;
    const int tid = threadIdx.x, l = tid % TPL, gid = tid / TPL;
    constexpr unsigned m = 0xffffffffu;                      // every warp runs the loops below in step: whole-warp barriers
    static_assert((HP % C::NG == 0 || C::NG % HP == 0) && (QP % C::NG == 0 || C::NG % QP == 0), "whole warps take part in both loops");
    float2 *line = wbuf + gid * C::LS;
    load_plane_twiddles<LOG2P>(tw, twh, p.gtw, p.gtw_n, tid);
    __syncthreads();
    PlaneTw<LOG2P, true> twp;
    twp.init(l, tw, twh + HP, tid, kPlaneThreads);
    __syncthreads();
    const T *pq = (const T *)p.a;
    T *py = (T *)p.y;
    const T *pq2 = (const T *)p.q2;
    T *py2 = (T *)p.y2;
    const int Lx = p.lx, Ly = p.ly;
    const bool gated = pq != nullptr;                        // no gate tensor: the convolution itself is written (gate 1)
    const T qfill = gated ? T(0.f) : T(1.f);
    uint4 qvfill;
    {
        float f[Vec16<T>::VEC];
#pragma unroll
        for (int e = 0; e < Vec16<T>::VEC; ++e) f[e] = gated ? 0.f : 1.f;
        qvfill = Vec16<T>::pack(f);
    }
    for (long long pl = blockIdx.x; pl < p.planes; pl += gridDim.x) {
        const float2 *src = p.in + pl * (long long)C::XH * P;
        // Column kx + NG is requested (into registers) between the two passes of column kx: the loads
        // are in flight during the second pass and the stores, and the registers are free by then.
        static_assert(FI::NP == 2, "two-pass plans");
        using P0 = typename FI::template Pass<0>;
        float2 pre[P0::IPL][P0::R];
        auto fetch = [&](int kx) {
            const float2 *s = src + (long long)kx * P + l;
#pragma unroll
            for (int i = 0; i < P0::IPL; ++i)
#pragma unroll
                for (int r = 0; r < P0::R; ++r) {
                    HN_G(s + i * TPL + r * (P / P0::R), 8);
                    pre[i][r] = __ldcg(s + i * TPL + r * (P / P0::R));
                }
        };
        if (gid < HP) fetch(gid);
        if (gid == 0) {
            // column 0 packs bins kx = 0 and kx = P/2: line 0 + i * line P/2, combined as the values arrive; the
            // transform itself is the same code for every column, so the group sharing this warp is not held up
            const float2 *sn = src + (long long)HP * P + l;
#pragma unroll
            for (int i = 0; i < P0::IPL; ++i)
#pragma unroll
                for (int r = 0; r < P0::R; ++r) {
                    HN_G(sn + i * TPL + r * (P / P0::R), 8);
                    const float2 gn = __ldcg(sn + i * TPL + r * (P / P0::R));
                    pre[i][r] = make_float2(pre[i][r].x - gn.y, pre[i][r].y + gn.x);
                }
        }
        // Rows y and y + P/4 leave as one complex row transform (real part row y, imaginary part row y + P/4).  With A, B
        // the values of column kx at the two rows, that transform's input is G[kx] = A + iB at bin kx and
        // G[P - kx] = conj A + i conj B at the mirrored bin: the column transform forms both from its last pass's
        // registers (legs r and r + R/4 of a lane are a row pair) and stores the whole line G of every row pair, so the
        // row transform loads one value per point.  The packed column (kx = 0 with kx = P/2) stores the same two
        // combinations at bins 0 and P/2; the row phase turns them into (A.x, B.x) and (A.y, B.y).
        using P1 = typename FI::template Pass<1>;
        for (int kx = gid; kx < HP; kx += C::NG) {
            float2 *lo = cs + kx * CSI, *hi = cs + (kx == 0 ? HP : P - kx) * CSI;
            FI::template pass<0, PRUNE_NONE>(l, twp,
                [&](int i, int r, int) { return pre[i][r]; },
                [&](int, int, int idx, float2 v) { line[FI::ph(idx)] = v; });
            __syncwarp(m);
            if (kx + C::NG < HP) fetch(kx + C::NG);
            float2 first[P1::IPL][P1::R / 4];
            FI::template pass<1, PRUNE_OUT>(l, twp,
                [&](int, int, int idx) { return line[FI::ph(idx)]; },
                [&](int i, int r, int idx, float2 B) {
                    if (r < P1::R / 4) { first[i][r] = B; return; }
                    const float2 A = first[i][r - P1::R / 4];
                    lo[idx - QP] = make_float2(A.x - B.y, A.y + B.x);
                    hi[idx - QP] = make_float2(A.x + B.y, B.x - A.y);
                });
            __syncwarp(m);
        }
        // The gate values of all of this lane's outputs are requested before anything else of the row phase (before
        // the barrier, and before the prefetch below, whose burst of requests would otherwise sit in front of them).
        const long long ob = pl * (long long)Ly * Lx;
        using PE = typename FI::LastPass;
        constexpr int NQ = PE::IPL * (PE::R / 2);
        constexpr int RIT = QP > C::NG ? QP / C::NG : 1;      // row pairs per lane group
        constexpr int VEC = Vec16<T>::VEC, NV = (HP / VEC + TPL - 1) / TPL;      // vectors per row and lane
        T q0[VST ? 1 : RIT][VST ? 1 : NQ], q1[VST ? 1 : RIT][VST ? 1 : NQ];
        uint4 qv0[VST ? RIT : 1][VST ? NV : 1], qv1[VST ? RIT : 1][VST ? NV : 1];
#pragma unroll
        for (int it = 0; it < RIT; ++it) {
            const int rp = gid + it * C::NG, y1 = rp + QP;
            const bool has0 = rp < QP, has1 = has0 && y1 < Ly;
            const long long o0 = ob + (long long)rp * Lx, o1 = ob + (long long)y1 * Lx;
            if constexpr (VST) {
#pragma unroll
                for (int j = 0; j < NV; ++j) {
                    const int x0 = (l + j * TPL) * VEC;
                    qv0[it][j] = qv1[it][j] = qvfill;
                    if (x0 < Lx && has0 && gated) { HN_G(pq + o0 + x0, 16); qv0[it][j] = __ldg(reinterpret_cast<const uint4 *>(pq + o0 + x0)); }
                    if (x0 < Lx && has1 && gated) { HN_G(pq + o1 + x0, 16); qv1[it][j] = __ldg(reinterpret_cast<const uint4 *>(pq + o1 + x0)); }
                }
            } else {
#pragma unroll
                for (int i = 0; i < PE::IPL; ++i)
#pragma unroll
                    for (int r = 0; r < PE::R / 2; ++r) {
                        const int idx = FI::last_pos(l, i, r);
                        if (idx < Lx && has0 && gated) HN_G(pq + o0 + idx, sizeof(T));
                        if (idx < Lx && has1 && gated) HN_G(pq + o1 + idx, sizeof(T));
                        q0[it][i * (PE::R / 2) + r] = (idx < Lx && has0 && gated) ? __ldg(pq + o0 + idx) : qfill;
                        q1[it][i * (PE::R / 2) + r] = (idx < Lx && has1 && gated) ? __ldg(pq + o1 + idx) : qfill;
                    }
            }
        }
        __syncthreads();
        if (pl + gridDim.x < p.planes) {
            // while the rows are transformed, bring the next plane's spectra and gate into L2
            prefetch_l2(p.in + (pl + gridDim.x) * (long long)C::XH * P, (long long)C::XH * P * sizeof(float2), tid);
            if (gated) prefetch_l2(pq + (pl + gridDim.x) * (long long)Ly * Lx, (long long)Ly * Lx * sizeof(T), tid);
        }
#pragma unroll
        for (int it = 0; it < RIT; ++it) {
            const int rp = gid + it * C::NG;
            if (rp >= QP) break;
            const int y1 = rp + QP;
            const bool has1 = y1 < Ly;
            const long long o0 = ob + (long long)rp * Lx, o1 = ob + (long long)y1 * Lx;
            static_assert(P0::IPL == 1, "lane 0 holds bins 0 and P/2 of a row");
            const float2 *g = cs + l * CSI + rp;
            float2 nyq = make_float2(0.f, 0.f);
            auto spectrum = [&](int, int r, int) {
                    float2 v = g[r * (P / P0::R) * CSI];
                    if (r == 0 && l == 0) {
                        // bins 0 and P/2 hold A + iB and conj A + i conj B of the packed column, A = (X_0[y], X_{P/2}[y]):
                        // the row transform wants (A.x, B.x) at bin 0 and (A.y, B.y) at bin P/2
                        const float2 w = g[HP * CSI];
                        nyq = make_float2(0.5f * (v.y - w.y), 0.5f * (w.x - v.x));
                        v = make_float2(0.5f * (v.x + w.x), 0.5f * (v.y + w.y));
                    }
                    if (r == P0::R / 2 && l == 0) v = nyq;
                    return v;
                };
            if constexpr (VST) {
                // results to the line in natural order; a lane then takes VEC neighbouring outputs of both rows
                FI::template run_to_line<PRUNE_OUT>(l, m, twp, line, spectrum);
#pragma unroll
                for (int j = 0; j < NV; ++j) {
                    const int x0 = (l + j * TPL) * VEC;
                    if (x0 < Lx) {
                        float a[VEC], b[VEC], ga[VEC], gb[VEC];
                        Vec16<T>::unpack(qv0[it][j], ga);
                        Vec16<T>::unpack(qv1[it][j], gb);
#pragma unroll
                        for (int e = 0; e < VEC; ++e) {
                            const float2 z = line[FI::ph(x0 + e)];
                            a[e] = z.x * ga[e];
                            b[e] = z.y * gb[e];
                        }
                        HN_G(py + o0 + x0, 16);
                        *reinterpret_cast<uint4 *>(py + o0 + x0) = Vec16<T>::pack(a);
                        if (has1) { HN_G(py + o1 + x0, 16); *reinterpret_cast<uint4 *>(py + o1 + x0) = Vec16<T>::pack(b); }
                    }
                }
                if constexpr (TWO) {
#pragma unroll
                    for (int j = 0; j < NV; ++j) {
                        const int x0 = (l + j * TPL) * VEC;
                        if (x0 < Lx) {
                            float a[VEC], b[VEC], ga[VEC], gb[VEC];
                            HN_G(pq2 + o0 + x0, 16);
                            Vec16<T>::unpack(__ldg(reinterpret_cast<const uint4 *>(pq2 + o0 + x0)), ga);
                            if (has1) HN_G(pq2 + o1 + x0, 16);
                            Vec16<T>::unpack(has1 ? __ldg(reinterpret_cast<const uint4 *>(pq2 + o1 + x0)) : make_uint4(0u, 0u, 0u, 0u), gb);
#pragma unroll
                            for (int e = 0; e < VEC; ++e) {
                                const float2 z = line[FI::ph(x0 + e)];
                                a[e] = z.x * ga[e];
                                b[e] = z.y * gb[e];
                            }
                            HN_G(py2 + o0 + x0, 16);
                            *reinterpret_cast<uint4 *>(py2 + o0 + x0) = Vec16<T>::pack(a);
                            if (has1) { HN_G(py2 + o1 + x0, 16); *reinterpret_cast<uint4 *>(py2 + o1 + x0) = Vec16<T>::pack(b); }
                        }
                    }
                }
            } else {
                FI::template run<PRUNE_OUT>(l, m, twp, line, spectrum,
                    [&](int i, int r, int idx, float2 v) {
                        if (idx < Lx) {
                            IO<T>::st(py, o0 + idx, v.x * (float)q0[it][i * (PE::R / 2) + r]);
                            if (has1) IO<T>::st(py, o1 + idx, v.y * (float)q1[it][i * (PE::R / 2) + r]);
                            if constexpr (TWO) {
                                IO<T>::st(py2, o0 + idx, v.x * IO<T>::ld(pq2, o0 + idx));
                                if (has1) IO<T>::st(py2, o1 + idx, v.y * IO<T>::ld(pq2, o1 + idx));
                            }
                        }
                    });
            }
            __syncwarp(m);
        }
        __syncthreads();
    }
}

// ---- launchers --------------------------------------------------------------------------------------------

static int plane_sms()
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

int plane_grid(long long planes)
{
    const int s = plane_sms();
    return (int)(planes < s ? planes : s);
}

template <typename T, int LOG2P> static int launch_plane_t(const PlaneArgs &a, int which, cudaStream_t st)
{
    using C = PlaneCfg<LOG2P>;
    const int grid = plane_grid(a.planes);
    if (grid <= 0) return 0;
    static DevOnce attr[6];
    // 16-byte gate loads and result stores where every row is a whole number of vectors on a 16-byte boundary
    const bool two = which == PLANE_INV && a.q2 != nullptr && a.y2 != nullptr;
    const bool vst = which == PLANE_INV && a.lx % Vec16<T>::VEC == 0 &&
                     (((uintptr_t)a.a | (uintptr_t)a.y | (uintptr_t)a.q2 | (uintptr_t)a.y2) & 15) == 0;
    void (*fn)(PlaneArgs) = which == PLANE_U ? uplane_kernel<T, LOG2P>
                          : which == PLANE_H ? hplane_kernel<T, LOG2P>
                          : two ? (vst ? plane_inv_kernel<T, LOG2P, true, true> : plane_inv_kernel<T, LOG2P, false, true>)
                                : (vst ? plane_inv_kernel<T, LOG2P, true, false> : plane_inv_kernel<T, LOG2P, false, false>);
    if (vst) which = 3;
    if (two) which = vst ? 5 : 4;
    if (attr[which].first()) {
        cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)C::SMEM);
    }
    fn<<<grid, kPlaneThreads, C::SMEM, st>>>(a);
    return 1;
}

int launch_plane(const PlaneArgs &a, int which, int log2p, int dtype, cudaStream_t st)
{
    if (log2p == 8) return dtype == 0 ? launch_plane_t<float, 8>(a, which, st) : launch_plane_t<bf16, 8>(a, which, st);
    if (log2p == 7) return dtype == 0 ? launch_plane_t<float, 7>(a, which, st) : launch_plane_t<bf16, 7>(a, which, st);
    return -1;
}

bool plane_supported(int log2p) { return log2p == 7 || log2p == 8; }

}  // namespace hn
