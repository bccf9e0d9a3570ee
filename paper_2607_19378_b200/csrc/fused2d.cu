// Fused 2-D path: the whole operator for one (b,c) slice in one CTA, nothing but
// q, k, v, h, y touches HBM (the single-stage kernel the paper's Appendix B.4 names
// as its goal for 2-D; its published pipeline still uses three kernels).
//
// Per slice: rows of the filter and of k*v are transformed two real rows per complex transform
// (rows y and y + P/2 of the filter, y and y + P/4 of k*v) and the raw transforms go straight
// into shared-memory stores [bin][row pair]; every column kx = 0 .. P/2 then runs
//   forward(filter column) -> registers, forward(k*v column), product (Eq. 12),
//   inverse, keep the cropped half
// in one group of lanes, separating the two real rows of each pair as it loads
//   2 F_y[kx] = Z[kx] + conj Z[P - kx],   2 F_y'[kx] = -i (Z[kx] - conj Z[P - kx])
// and combining two result rows into one complex row G = A + iB (bin kx) and conj A + i conj B
// (bin P - kx) as it stores, in place: bins kx and P - kx of the k*v store belong to column kx
// alone.  Finally the rows are transformed back (one load per point), cropped, gated by q and
// stored.  Used when both padded axes are equal and at most 128 points.
#include "common.cuh"
#include "fused2d.cuh"
#include "plane_util.cuh"

namespace hn {

constexpr int kF2Threads = kPlaneThreads + 32;               // 68 groups of 8 lanes: one per column kx = 0 .. 64 of a 128-point plane

template <int LOG2P> struct F2Cfg {
    static constexpr int P = 1 << LOG2P, HP = P / 2, QP = P / 4;
    static constexpr int HCS = HP + 1;                       // filter store stride (odd): P bins of P/2 row pairs
    static constexpr int UCS = QP + 1;                       // k*v store stride (odd): P bins of P/4 row pairs
    using F = WF<LOG2P, false>;
    using FI = WF<LOG2P, true>;
    static constexpr int NGM = kPlaneThreads / F::TPL;       // groups of the 16 main warps
    static constexpr int NG = kF2Threads / F::TPL;           // all groups
    static constexpr int LS = plane_ls(P);
    // entries per store, rounded to an even count: what follows them (the lines, which receive 16-byte
    // asynchronous copies) must start on a 16-byte boundary
    static constexpr int HCSN = (P * HCS + 1) & ~1, UCSN = (P * UCS + 1) & ~1;
    static constexpr size_t SMEM = sizeof(float2) * ((size_t)HCSN + 2 * (size_t)UCSN + (size_t)NG * LS + 3 * P);
};

// Schedule per CTA (slices s0, s1, ... of this CTA):
//   phase 1  all main groups: filter rows of s_i; then half of them k*v rows of s_i while the other
//            half turns the finished columns of s_(i-1) back into rows, crops, gates and stores
//   phase 2  one group per column kx = 0 .. P/2 (the extra warp takes the last one); columns 0 and P/2 hold
//            real data and run as general complex transforms, which keeps all groups on one code path
// so every phase keeps all groups busy; the k*v store is double buffered.
// VST: rows are whole numbers of 16-byte vectors and q, y are 16-byte aligned: gate values arrive as 16-byte loads, the
// cropped rows go through the line once more and leave as 16-byte stores; else one element per lane and leg.
// TWO: a second gate and result, y2 = q2 * (the same convolution) (the backward pass: dk = v du and dv = k du).
template <typename T, int LOG2P, bool VST, bool TWO>
__global__ void __launch_bounds__(kF2Threads, 1) fused2d_kernel(Fused2dArgs p)     // 96 registers: one scheduler hosts 5 of the 17 warps
{
    using C = F2Cfg<LOG2P>;
    using F = typename C::F;
    using FI = typename C::FI;
    constexpr int P = C::P, HP = C::HP, QP = C::QP, TPL = F::TPL, NP = F::NP, NGM = C::NGM;
    constexpr int HCS = C::HCS, UCS = C::UCS;
    extern __shared__ float2 smem[];
    float2 *hcs = smem;
    static_assert((C::HCSN + 2 * C::UCSN) % 2 == 0 && C::LS % 2 == 0, "lines start on 16-byte boundaries");
    float2 *ucs0 = hcs + C::HCSN;
    float2 *wbuf = ucs0 + 2 * C::UCSN;
    float2 *tw = wbuf + C::NG * C::LS;
    const int tid = threadIdx.x, l = tid % TPL, gid = tid / TPL;
    const unsigned m = F::group_mask(tid);
    float2 *line = wbuf + gid * C::LS;
    for (int t = tid; t < P; t += kF2Threads) { HN_G(p.gtw + t * (p.gtw_n >> LOG2P), 8); tw[t] = p.gtw[t * (p.gtw_n >> LOG2P)]; }
    __syncthreads();
    PlaneTw<LOG2P, false> twf;
    twf.init(l, tw, tw + P, tid, kF2Threads);
    PlaneTw<LOG2P, true> twi;
    twi.init(l, tw, tw + 2 * P, tid, kF2Threads);
    __syncthreads();
    const unsigned char *kb = (const unsigned char *)p.k, *vb = (const unsigned char *)p.v;
    const unsigned char *hb = (const unsigned char *)p.h;
    const unsigned char *ke = kb + p.kv_elems * sizeof(T), *ve = vb + p.kv_elems * sizeof(T), *he = hb + p.h_elems * sizeof(T);
    const T *pq = (const T *)p.q;
    T *py = (T *)p.y;
    const T *pq2 = (const T *)p.q2;
    T *py2 = (T *)p.y2;
    const int Lx = p.lx, Ly = p.ly, Kx = 2 * Lx - 1, Ky = 2 * Ly - 1;
    const long long vol = (long long)Lx * Ly, kvol = (long long)Kx * Ky;
    using PL = typename F::LastPass;
    using PF0 = typename F::template Pass<0>;
    using PI0 = typename FI::template Pass<0>;
    using PIL = typename FI::LastPass;
    constexpr int ES = (int)sizeof(T);
    const int J0 = HP + 1 - Lx;                              // window position of filter tap 0 (see below)
    const int RU = (J0 * ES + 15) & ~15;                     // bytes kept free before the first copied chunk
    const float sc = 0.25f * p.scale;                        // the two separations leave a factor 2 each

    // rows back for slice sp, reading the store ub (lines G of the row pairs); groups g0, g0 + gstep, ... take part
    auto rows_back = [&](long long sp, const float2 *ub, int g0, int gstep) {
        for (int rp = spread_pair<8>(g0); rp < QP; rp += gstep) {
            const int y1 = rp + QP;
            const bool has1 = y1 < Ly;
            const long long o0 = sp * vol + (long long)rp * Lx, o1 = sp * vol + (long long)y1 * Lx;
            // the gate values of this lane's outputs are requested before the transform starts
            constexpr int NQ = PIL::IPL * (PIL::R / 2);
            constexpr int VEC = Vec16<T>::VEC, NV = (HP / VEC + TPL - 1) / TPL;       // vectors per row and lane
            const float2 *g = ub + l * UCS + rp;
            auto spectrum = [&](int i, int r, int) { return g[(i * TPL + r * (P / PI0::R)) * UCS]; };
            if constexpr (VST) {
                uint4 qv0[NV], qv1[NV];
#pragma unroll
                for (int j = 0; j < NV; ++j) {
                    const int x0 = (l + j * TPL) * VEC;
                    qv0[j] = qv1[j] = make_uint4(0u, 0u, 0u, 0u);
                    if (x0 < Lx) { HN_G(pq + o0 + x0, 16); qv0[j] = __ldg(reinterpret_cast<const uint4 *>(pq + o0 + x0)); }
                    if (x0 < Lx && has1) { HN_G(pq + o1 + x0, 16); qv1[j] = __ldg(reinterpret_cast<const uint4 *>(pq + o1 + x0)); }
                }
                FI::template run_to_line<PRUNE_OUT>(l, m, twi, line, spectrum);
#pragma unroll
                for (int j = 0; j < NV; ++j) {
                    const int x0 = (l + j * TPL) * VEC;
                    if (x0 < Lx) {
                        float a[VEC], b[VEC], ga[VEC], gb[VEC];
                        Vec16<T>::unpack(qv0[j], ga);
                        Vec16<T>::unpack(qv1[j], gb);
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
                T q0[NQ], q1[NQ];
#pragma unroll
                for (int i = 0; i < PIL::IPL; ++i)
#pragma unroll
                    for (int r = 0; r < PIL::R / 2; ++r) {
                        const int idx = FI::last_pos(l, i, r);
                        if (idx < Lx) HN_G(pq + o0 + idx, ES);
                        if (idx < Lx && has1) HN_G(pq + o1 + idx, ES);
                        q0[i * (PIL::R / 2) + r] = idx < Lx ? __ldg(pq + o0 + idx) : T(0.f);
                        q1[i * (PIL::R / 2) + r] = (idx < Lx && has1) ? __ldg(pq + o1 + idx) : T(0.f);
                    }
                FI::template run<PRUNE_OUT>(l, m, twi, line, spectrum,
                    [&](int i, int r, int idx, float2 v) {
                        if (idx < Lx) {
                            IO<T>::st(py, o0 + idx, v.x * (float)q0[i * (PIL::R / 2) + r]);
                            if (has1) IO<T>::st(py, o1 + idx, v.y * (float)q1[i * (PIL::R / 2) + r]);
                            if constexpr (TWO) {
                                HN_G(pq2 + o0 + idx, ES);
                                IO<T>::st(py2, o0 + idx, v.x * IO<T>::ld(pq2, o0 + idx));
                                if (has1) { HN_G(pq2 + o1 + idx, ES); IO<T>::st(py2, o1 + idx, v.y * IO<T>::ld(pq2, o1 + idx)); }
                            }
                        }
                    });
            }
            __syncwarp(m);
        }
    };

    int cur = 0;
    long long sprev = -1;
    for (long long s = blockIdx.x; s < p.slices; s += gridDim.x) {
        float2 *ucs = ucs0 + cur * C::UCSN;
        const long long hs = p.h_mod ? (s + p.h_off) % p.h_mod : s;
        if (gid < NGM) {
            // ---- filter rows: padded row yp holds tap row (yp + Ly - 1) mod P; rows yp and yp + P/2 share a transform
            // (at most one of the two lies in the zero band, which is shorter than P/2 rows).  Padded position x of a
            // row holds tap (x + Lx - 1) mod P, so the P positions are a window W of P consecutive tap indices starting
            // at -(P/2 + 1 - Lx), zeros outside [0, Kx): position x is W[x + P/2], position x + P/2 is W[x] (x < P/2);
            // a thread's taps sit at constant offsets from one address.
            for (int rp = spread_pair<8>(gid); rp < HP; rp += NGM) {
                const int my0 = (rp + Ly - 1) & (P - 1), my1 = my0 ^ HP;
                const bool v0 = my0 < Ky, v1 = my1 < Ky;
                constexpr int SLOT = P * ES + 48;            // window, alignment slack, last chunk
                static_assert(2 * SLOT + 32 <= C::LS * 8, "staged rows must fit the line");
                // lines 2 and 3 of a warp stage 32 bytes further in: the narrow tap loads of the four lines
                // then use different banks
                unsigned char *s0 = reinterpret_cast<unsigned char *>(line) + 16 * (gid & 2), *s1 = s0 + SLOT;
                const unsigned char *g0 = hb + (hs * kvol + (long long)my0 * Kx) * ES;
                const unsigned char *g1 = hb + (hs * kvol + (long long)my1 * Kx) * ES;
                const int n0 = v0 ? Kx : 0, n1 = v1 ? Kx : 0;
                if (v0) stage_row_u<TPL, (P - 1) * ES>(s0 + RU, g0, Kx * ES, hb, he, l);
                if (v1) stage_row_u<TPL, (P - 1) * ES>(s1 + RU, g1, Kx * ES, hb, he, l);
                cp_async_wait_all();
                __syncwarp(m);
                // window element j sits at w + j * ES; blank what lies outside the row once
                unsigned char *w0 = s0 + RU + (int)((unsigned long long)g0 & 15ull) - J0 * ES;
                unsigned char *w1 = s1 + RU + (int)((unsigned long long)g1 & 15ull) - J0 * ES;
                for (int j = l; j < J0; j += TPL) {
                    *reinterpret_cast<T *>(w0 + j * ES) = T(0.f);
                    *reinterpret_cast<T *>(w1 + j * ES) = T(0.f);
                }
                for (int j = J0 + n0 + l; j < P; j += TPL) *reinterpret_cast<T *>(w0 + j * ES) = T(0.f);
                for (int j = J0 + n1 + l; j < P; j += TPL) *reinterpret_cast<T *>(w1 + j * ES) = T(0.f);
                __syncwarp(m);
                const T *t0 = reinterpret_cast<const T *>(w0) + l, *t1 = reinterpret_cast<const T *>(w1) + l;
                F::template run<PRUNE_NONE, true>(l, m, twf, line,
                    [&](int i, int r, int) {
                        const int x = i * TPL + r * (P / PF0::R);               // + l: padded position
                        const int j = r < PF0::R / 2 ? x + HP : x - HP;          // its window element
                        return make_float2((float)t0[j], (float)t1[j]);
                    },
                    [&](int, int, int kk, float2 z) { hcs[kk * HCS + rp] = z; });
                __syncwarp(m);
            }
            if (gid < NGM / 2) {
                // ---- k*v rows of this slice: y and y + P/4 share a transform (a missing partner is a zero row) ----
                for (int rp = spread_pair<8>(gid); rp < QP; rp += NGM / 2) {
                    const int y1 = rp + QP;
                    const bool has1 = y1 < Ly;
                    constexpr int SLOT = HP * ES + 32;
                    static_assert(4 * SLOT <= C::LS * 8, "staged rows must fit the line");
                    unsigned char *sk0 = reinterpret_cast<unsigned char *>(line), *sk1 = sk0 + SLOT, *sv0 = sk1 + SLOT, *sv1 = sv0 + SLOT;
                    const int rowb = Lx * ES;
                    const unsigned char *gk0 = kb + (s * vol + (long long)rp * Lx) * ES, *gk1 = gk0 + (long long)QP * rowb;
                    const unsigned char *gv0 = vb + (s * vol + (long long)rp * Lx) * ES, *gv1 = gv0 + (long long)QP * rowb;
                    stage_row_u<TPL, HP * ES>(sk0, gk0, rowb, kb, ke, l);
                    stage_row_u<TPL, HP * ES>(sv0, gv0, rowb, vb, ve, l);
                    if (has1) {
                        stage_row_u<TPL, HP * ES>(sk1, gk1, rowb, kb, ke, l);
                        stage_row_u<TPL, HP * ES>(sv1, gv1, rowb, vb, ve, l);
                    }
                    cp_async_wait_all();
                    __syncwarp(m);
                    const T *k0 = reinterpret_cast<const T *>(sk0 + ((unsigned long long)gk0 & 15ull)) + l;
                    const T *v0p = reinterpret_cast<const T *>(sv0 + ((unsigned long long)gv0 & 15ull)) + l;
                    const T *k1 = reinterpret_cast<const T *>(sk1 + ((unsigned long long)gk1 & 15ull)) + l;
                    const T *v1p = reinterpret_cast<const T *>(sv1 + ((unsigned long long)gv1 & 15ull)) + l;
                    auto keep = [&](int, int, int kk, float2 z) { ucs[kk * UCS + rp] = z; };
                    if (Lx == HP && has1) {
                        // full rows: no bounds tests in the input functor
                        F::template run<PRUNE_IN, true>(l, m, twf, line, [&](int i, int r, int) {
                            const int x = i * TPL + r * (P / PF0::R);
                            return make_float2((float)k0[x] * (float)v0p[x], (float)k1[x] * (float)v1p[x]);
                        }, keep);
                    } else {
                        F::template run<PRUNE_IN, true>(l, m, twf, line, [&](int i, int r, int idx) {
                            const int x = i * TPL + r * (P / PF0::R);
                            float a = 0.f, b = 0.f;
                            if (idx < Lx) {
                                a = (float)k0[x] * (float)v0p[x];
                                if (has1) b = (float)k1[x] * (float)v1p[x];
                            }
                            return make_float2(a, b);
                        }, keep);
                    }
                    __syncwarp(m);
                }
            } else if (sprev >= 0) {
                // ---- rows back of the previous slice (its columns were finished last iteration) ----
                rows_back(sprev, ucs0 + (cur ^ 1) * C::UCSN, gid - NGM / 2, NGM / 2);
            }
        }
        __syncthreads();
        {
            // the next slice's tensors travel to L2 during the column phase, which loads nothing from global memory
            const long long sn = s + gridDim.x;
            if (sn < p.slices && tid < kPlaneThreads) {
                const long long hn2 = p.h_mod ? (sn + p.h_off) % p.h_mod : sn;
                prefetch_l2(hb + hn2 * kvol * ES, kvol * ES, tid);
                prefetch_l2(kb + sn * vol * ES, vol * ES, tid);
                prefetch_l2(vb + sn * vol * ES, vol * ES, tid);
                prefetch_l2(pq + sn * vol, vol * ES, tid);
            }
        }
        // ---- columns: filter spectrum, k*v spectrum, product, inverse --------------------------
        for (int kx = spread_pair<8>(gid); kx <= HP; kx += C::NG) {
            const int km = (P - kx) & (P - 1);
            const float2 *ha = hcs + kx * HCS, *hm = hcs + km * HCS;
            float2 *ua = ucs + kx * UCS, *um = ucs + km * UCS;
            float2 H[PL::IPL][PL::R];
            {
                float2 second[PF0::IPL][PF0::R / 2] = {};     // rows y + P/2, formed with their partners y
                F::template run<PRUNE_NONE>(l, m, twf, line,
                    [&](int i, int r, int idx) {
                        if (r >= PF0::R / 2) return second[i][r - PF0::R / 2];
                        const float2 za = ha[idx], zm = hm[idx];
                        second[i][r] = make_float2(za.y + zm.y, zm.x - za.x);
                        return make_float2(za.x + zm.x, za.y - zm.y);
                    },
                    [&](int i, int r, int, float2 v) { H[i][r] = make_float2(v.x * sc, v.y * sc); });
            }
            __syncwarp(m);
            float2 Y[PL::IPL][PL::R];
            {
                float2 second[PF0::IPL][PF0::R / 4] = {};     // rows y + P/4 (the upper half of the column is padding)
                F::template run<PRUNE_IN>(l, m, twf, line,
                    [&](int i, int r, int idx) {
                        if (r >= PF0::R / 4) return second[i][r - PF0::R / 4];
                        const float2 za = ua[idx], zm = um[idx];
                        second[i][r] = make_float2(za.y + zm.y, zm.x - za.x);
                        return make_float2(za.x + zm.x, za.y - zm.y);
                    },
                    [&](int i, int r, int, float2 v) { Y[i][r] = cmul(v, H[i][r]); });
            }
            __syncwarp(m);
            FI::template pass<0, PRUNE_NONE>(l, twi,
                [&](int i, int r, int) { return Y[i][r]; },
                [&](int, int, int idx, float2 v) { line[FI::ph(idx)] = v; });
            __syncwarp(m);
            FI::template mid<1, NP - 1, PRUNE_NONE>(l, m, twi, line);
            // rows y and y + P/4 of the result leave as one complex row: G[kx] = A + iB, G[P - kx] = conj A + i conj B
            // (for the real columns kx = 0 and kx = P/2 the two coincide)
            const bool two = kx != 0 && kx != HP;
            float2 first[PIL::IPL][PIL::R / 4];
            FI::template pass<NP - 1, PRUNE_OUT>(l, twi,
                [&](int, int, int idx) { return line[FI::ph(idx)]; },
                [&](int i, int r, int idx, float2 B) {
                    if (r < PIL::R / 4) { first[i][r] = B; return; }
                    const float2 A = first[i][r - PIL::R / 4];
                    ua[idx - QP] = make_float2(A.x - B.y, A.y + B.x);
                    if (two) um[idx - QP] = make_float2(A.x + B.y, B.x - A.y);
                });
            __syncwarp(m);
        }
        __syncthreads();
        sprev = s;
        cur ^= 1;
    }
    if (sprev >= 0 && gid < NGM) rows_back(sprev, ucs0 + (cur ^ 1) * C::UCSN, gid, NGM);
}

template <typename T, int LOG2P> static int launch_fused2d_t(const Fused2dArgs &a, cudaStream_t st)
{
    using C = F2Cfg<LOG2P>;
    static int sms = 0;
    if (!sms) {
        int dev = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (sms <= 0) sms = 148;
    }
    // 16-byte gate loads and result stores where every row is a whole number of vectors on a 16-byte boundary
    const bool two = a.q2 != nullptr && a.y2 != nullptr;
    const bool vst = a.lx % Vec16<T>::VEC == 0 &&
                     (((uintptr_t)a.q | (uintptr_t)a.y | (uintptr_t)a.q2 | (uintptr_t)a.y2) & 15) == 0;
    static DevOnce attr[4];
    void (*fn)(Fused2dArgs) = two ? (vst ? fused2d_kernel<T, LOG2P, true, true> : fused2d_kernel<T, LOG2P, false, true>)
                                  : (vst ? fused2d_kernel<T, LOG2P, true, false> : fused2d_kernel<T, LOG2P, false, false>);
    if (attr[(two ? 2 : 0) + (vst ? 1 : 0)].first()) cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)C::SMEM);
    const int grid = (int)(a.slices < sms ? a.slices : sms);
    if (grid <= 0) return 0;
    fn<<<grid, kF2Threads, C::SMEM, st>>>(a);
    return 1;
}

bool fused2d_supported(int log2p) { return log2p == 6 || log2p == 7; }

int launch_fused2d(const Fused2dArgs &a, int log2p, int dtype, cudaStream_t st)
{
    if (log2p == 7) return dtype == 0 ? launch_fused2d_t<float, 7>(a, st) : launch_fused2d_t<bf16, 7>(a, st);
    if (log2p == 6) return dtype == 0 ? launch_fused2d_t<float, 6>(a, st) : launch_fused2d_t<bf16, 6>(a, st);
    return -1;
}

}  // namespace hn
