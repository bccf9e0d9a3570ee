// Fused 2-D path: the whole operator for one (b,c) slice in one CTA, nothing but
// q, k, v, h, y touches HBM (the single-stage kernel the paper's Appendix B.4 names
// as its goal for 2-D; its published pipeline still uses three kernels).
//
// Per slice: rows of the filter and of k*v are transformed two real rows per complex
// transform and scattered into shared-memory column stores (half spectra, with the two
// purely real bins of a row packed into column 0); every column then runs
//   forward(filter column) -> registers, forward(k*v column), product (Eq. 12),
//   inverse, keep the cropped half
// in one group of lanes; finally the rows are transformed back, cropped, gated by q
// and stored.  Used when both padded axes are equal and at most 128 points.
#include "common.cuh"
#include "fused2d.cuh"
#include "plane_util.cuh"

namespace hn {

constexpr int kF2Threads = kPlaneThreads + 32;               // 68 groups of 8 lanes: one per column kx = 0 .. 64 of a 128-point plane

template <int LOG2P> struct F2Cfg {
    static constexpr int P = 1 << LOG2P, HP = P / 2;
    static constexpr int HCSS = P + 1;                       // filter column store stride (odd)
    static constexpr int UCSS = HP + 1;                      // k*v column store stride (odd)
    using F = WF<LOG2P, false>;
    using FI = WF<LOG2P, true>;
    static constexpr int NGM = kPlaneThreads / F::TPL;       // groups of the 16 main warps
    static constexpr int NG = kF2Threads / F::TPL;           // all groups
    static constexpr int LS = plane_ls(P);
    static constexpr int NCOL = HP + 1;                      // columns kx = 0 .. P/2, none packed
    // entries per column store, rounded to an even count: what follows them (the lines, which receive 16-byte
    // asynchronous copies) must start on a 16-byte boundary
    static constexpr int HCSN = (NCOL * HCSS + 1) & ~1, UCSN = (NCOL * UCSS + 1) & ~1;
    static constexpr size_t SMEM = sizeof(float2) * ((size_t)HCSN + 2 * (size_t)UCSN + (size_t)NG * LS + 3 * P);
};

// Schedule per CTA (slices s0, s1, ... of this CTA):
//   phase 1  all main groups: filter rows of s_i; then half of them k*v rows of s_i while the other
//            half turns the finished columns of s_(i-1) back into rows, crops, gates and stores
//   phase 2  main groups: one column each (filter spectrum -> registers, k*v spectrum, product,
//            inverse); the extra warp: the packed column (bins kx = 0 and kx = P/2), its filter part
//            and its k*v part on two groups side by side
// so every phase keeps all groups busy; the k*v column store is double buffered.
template <typename T, int LOG2P>
__global__ void __launch_bounds__(kF2Threads, 1) fused2d_kernel(Fused2dArgs p)
{
    using C = F2Cfg<LOG2P>;
    using F = typename C::F;
    using FI = typename C::FI;
    constexpr int P = C::P, HP = C::HP, TPL = F::TPL, NP = F::NP, NGM = C::NGM;
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
    const T *pq = (const T *)p.q;
    T *py = (T *)p.y;
    const int Lx = p.lx, Ly = p.ly, Kx = 2 * Lx - 1, Ky = 2 * Ly - 1;
    const long long vol = (long long)Lx * Ly, kvol = (long long)Kx * Ky;
    using PL = typename F::LastPass;

    // rows back for slice sp, reading column store ub; groups g0, g0 + gstep, ... take part
    auto rows_back = [&](long long sp, const float2 *ub, int g0, int gstep) {
        for (int rp = spread_pair<4>(g0); 2 * rp < Ly; rp += gstep) {
            const int y0 = 2 * rp, y1 = y0 + 1;
            const bool has1 = y1 < Ly;
            const long long o0 = sp * vol + (long long)y0 * Lx, o1 = o0 + Lx;
            FI::template run<PRUNE_OUT>(l, m, twi, line,
                [&](int, int, int idx) {
                    // branch-free merge of two half spectra into one complex row
                    const bool mirror = idx > HP;
                    const int kx = mirror ? P - idx : idx;
                    const float2 A = ub[kx * C::UCSS + y0];
                    float2 B = ub[kx * C::UCSS + y1];
                    if (!has1) B = make_float2(0.f, 0.f);
                    const float sg = mirror ? -1.f : 1.f;
                    return make_float2(fmaf(-sg, B.y, A.x), fmaf(sg, A.y, B.x));
                },
                [&](int, int, int idx, float2 v) {
                    if (idx < Lx) {
                        IO<T>::st(py, o0 + idx, v.x * IO<T>::ld(pq, o0 + idx));
                        if (has1) IO<T>::st(py, o1 + idx, v.y * IO<T>::ld(pq, o1 + idx));
                    }
                });
            __syncwarp(m);
        }
    };

    int cur = 0;
    long long sprev = -1;
    for (long long s = blockIdx.x; s < p.slices; s += gridDim.x) {
        float2 *ucs = ucs0 + cur * C::UCSN;
        const long long hs = p.h_mod ? (s + p.h_off) % p.h_mod : s;
        const long long sn = s + gridDim.x;
        if (sn < p.slices && tid < kPlaneThreads) {
            const long long hn2 = p.h_mod ? (sn + p.h_off) % p.h_mod : sn;
            prefetch_l2(hb + hn2 * kvol * sizeof(T), kvol * sizeof(T), tid);
            prefetch_l2(kb + sn * vol * sizeof(T), vol * sizeof(T), tid);
            prefetch_l2(vb + sn * vol * sizeof(T), vol * sizeof(T), tid);
            prefetch_l2(pq + sn * vol, vol * sizeof(T), tid);
        }
        if (gid < NGM) {
            // ---- filter rows: padded position yp holds tap my = (yp + Ly - 1) mod P ----------
            for (int rp = spread_pair<4>(gid); 2 * rp < P; rp += NGM) {
                const int yp0 = 2 * rp, yp1 = yp0 + 1;
                const int my0 = (yp0 + Ly - 1) & (P - 1), my1 = (yp1 + Ly - 1) & (P - 1);
                const bool v0 = my0 < Ky, v1 = my1 < Ky;
                if (v0 || v1) {
                    constexpr int SLOT = ((P - 1) * (int)sizeof(T) + 15) / 16 * 16 + 16;
                    static_assert(2 * SLOT + 32 <= C::LS * 8, "staged rows must fit the line");
                    // lines 2 and 3 of a warp stage 32 bytes further in: the narrow tap loads of the four lines
                    // then use different banks
                    unsigned char *s0 = reinterpret_cast<unsigned char *>(line) + 16 * (gid & 2), *s1 = s0 + SLOT;
                    const unsigned char *g0 = hb + (hs * kvol + (long long)my0 * Kx) * sizeof(T);
                    const unsigned char *g1 = hb + (hs * kvol + (long long)my1 * Kx) * sizeof(T);
                    if (v0) stage_row<TPL>(s0, g0, Kx * (int)sizeof(T), hb, hb + p.h_elems * sizeof(T), l);
                    if (v1) stage_row<TPL>(s1, g1, Kx * (int)sizeof(T), hb, hb + p.h_elems * sizeof(T), l);
                    cp_async_wait_all();
                    __syncwarp(m);
                    const int f0 = (int)((unsigned long long)g0 & 15ull), f1 = (int)((unsigned long long)g1 & 15ull);
                    // blank the padding taps (and a missing row) once: the input functor is branch-free
                    zero_staged<T, TPL>(s0, f0, v0 ? Kx : 0, P, l);
                    zero_staged<T, TPL>(s1, f1, v1 ? Kx : 0, P, l);
                    __syncwarp(m);
                    const int cw = (l + Lx - 1) & (P - 1);
                    F::template run_to_line<PRUNE_NONE, true>(l, m, twf, line, [&](int i, int r, int) {
                        const int mx = (cw + i * TPL + r * (P / F::template Pass<0>::R)) & (P - 1);
                        return make_float2(staged<T>(s0, f0, mx), staged<T>(s1, f1, mx));
                    });
                    separate_rows_full<LOG2P, C::HCSS>(line, hcs, yp0, yp1, l);
                    __syncwarp(m);
                } else {
                    for (int kx = l; kx <= HP; kx += TPL) {
                        hcs[kx * C::HCSS + yp0] = make_float2(0.f, 0.f);
                        hcs[kx * C::HCSS + yp1] = make_float2(0.f, 0.f);
                    }
                }
            }
            if (gid < NGM / 2) {
                // ---- k*v rows of this slice ---------------------------------------------------------
                for (int rp = spread_pair<4>(gid); 2 * rp < Ly; rp += NGM / 2) {
                    const int y0 = 2 * rp, y1 = y0 + 1;
                    const bool has1 = y1 < Ly;
                    const int nrow = (has1 ? 2 : 1) * Lx * (int)sizeof(T);
                    const unsigned char *gk = kb + (s * vol + (long long)y0 * Lx) * sizeof(T);
                    const unsigned char *gv = vb + (s * vol + (long long)y0 * Lx) * sizeof(T);
                    unsigned char *sk = reinterpret_cast<unsigned char *>(line);
                    unsigned char *sv = sk + C::LS * 4;
                    stage_row<TPL>(sk, gk, nrow, kb, kb + p.kv_elems * sizeof(T), l);
                    stage_row<TPL>(sv, gv, nrow, vb, vb + p.kv_elems * sizeof(T), l);
                    cp_async_wait_all();
                    __syncwarp(m);
                    const int ok = (int)((unsigned long long)gk & 15ull), ov = (int)((unsigned long long)gv & 15ull);
                    if (Lx == HP && has1) {
                        // full rows: no bounds tests in the input functor
                        F::template run_to_line<PRUNE_IN, true>(l, m, twf, line, [&](int, int, int idx) {
                            return make_float2(staged<T>(sk, ok, idx) * staged<T>(sv, ov, idx),
                                               staged<T>(sk, ok, HP + idx) * staged<T>(sv, ov, HP + idx));
                        });
                    } else {
                        F::template run_to_line<PRUNE_IN, true>(l, m, twf, line, [&](int, int, int idx) {
                            float a = 0.f, b = 0.f;
                            if (idx < Lx) {
                                a = staged<T>(sk, ok, idx) * staged<T>(sv, ov, idx);
                                if (has1) b = staged<T>(sk, ok, Lx + idx) * staged<T>(sv, ov, Lx + idx);
                            }
                            return make_float2(a, b);
                        });
                    }
                    separate_rows_full<LOG2P, C::UCSS>(line, ucs, y0, y1, l);
                    __syncwarp(m);
                }
            } else if (sprev >= 0) {
                // ---- rows back of the previous slice (its columns were finished last iteration) ----
                rows_back(sprev, ucs0 + (cur ^ 1) * C::UCSN, gid - NGM / 2, NGM / 2);
            }
        }
        __syncthreads();
        // ---- columns: filter spectrum, k*v spectrum, product, inverse --------------------------
        {
            // every column kx = 0 .. P/2 has a group of its own (columns 0 and P/2 hold real data: their
            // transforms are done as general complex ones, which keeps all groups on one code path)
            for (int kx = spread_pair<8>(gid); kx <= HP; kx += C::NG) {
                const float2 *hc = hcs + kx * C::HCSS;
                float2 *uc = ucs + kx * C::UCSS;
                float2 H[PL::IPL][PL::R];
                F::template run<PRUNE_NONE>(l, m, twf, line,
                    [&](int, int, int idx) { return hc[idx]; },
                    [&](int i, int r, int, float2 v) { H[i][r] = make_float2(v.x * p.scale, v.y * p.scale); });
                __syncwarp(m);
                float2 Y[PL::IPL][PL::R];
                F::template run<PRUNE_IN>(l, m, twf, line,
                    [&](int, int, int idx) { return idx < Ly ? uc[idx] : make_float2(0.f, 0.f); },
                    [&](int i, int r, int, float2 v) { Y[i][r] = cmul(v, H[i][r]); });
                __syncwarp(m);
                FI::template pass<0, PRUNE_NONE>(l, twi,
                    [&](int i, int r, int) { return Y[i][r]; },
                    [&](int, int, int idx, float2 v) { line[FI::ph(idx)] = v; });
                __syncwarp(m);
                FI::template mid<1, NP - 1, PRUNE_NONE>(l, m, twi, line);
                FI::template pass<NP - 1, PRUNE_OUT>(l, twi,
                    [&](int, int, int idx) { return line[FI::ph(idx)]; },
                    [&](int, int, int idx, float2 v) { uc[idx] = v; });
                __syncwarp(m);
            }
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
    static DevOnce attr;
    if (attr.first()) cudaFuncSetAttribute(fused2d_kernel<T, LOG2P>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)C::SMEM);
    const int grid = (int)(a.slices < sms ? a.slices : sms);
    if (grid <= 0) return 0;
    fused2d_kernel<T, LOG2P><<<grid, kF2Threads, C::SMEM, st>>>(a);
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
