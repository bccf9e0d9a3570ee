// Warp-local FFT engine: a group of TPL lanes (TPL <= 32) of one warp owns one
// line of N = 2^LOG2N complex points.  Each Stockham pass keeps R points per
// item in registers; passes are joined through a private shared-memory line
// and separated by __syncwarp() over the group's lanes only, so warps never wait for the rest of the
// CTA while transforming.  Inputs of the first pass and outputs of the last
// pass go through caller-supplied functors, which lets the callers read
// straight from global memory, zero-pad, gate, transpose, multiply spectra or
// chain a forward transform into an inverse one without extra round trips.
//
// The inverse uses the reversed radix sequence of the forward transform: the
// last forward pass then leaves, in each lane, exactly the points that lane
// needs for the first inverse pass (positions j + r*N/R), so the spectral
// product (Eq. 12 of the paper) happens in registers.
#pragma once
#include "fft_engine.cuh"

namespace hn {

template <int LOG2N> struct WPlan;
template <> struct WPlan<5>  { static constexpr int NP = 2, TPL = 4; static constexpr int R[3] = {8, 4, 1};
    __host__ __device__ static constexpr int r(int s) { return s == 0 ? 8 : s == 1 ? 4 : 1; } };
template <> struct WPlan<6>  { static constexpr int NP = 2, TPL = 8; static constexpr int R[3] = {8, 8, 1};
    __host__ __device__ static constexpr int r(int s) { return s == 0 ? 8 : s == 1 ? 8 : 1; } };
template <> struct WPlan<7>  { static constexpr int NP = 2, TPL = 8; static constexpr int R[3] = {8, 16, 1};
    __host__ __device__ static constexpr int r(int s) { return s == 0 ? 8 : s == 1 ? 16 : 1; } };
template <> struct WPlan<8>  { static constexpr int NP = 2, TPL = 16; static constexpr int R[3] = {16, 16, 1};
    __host__ __device__ static constexpr int r(int s) { return s == 0 ? 16 : s == 1 ? 16 : 1; } };
template <> struct WPlan<9>  { static constexpr int NP = 2, TPL = 16; static constexpr int R[3] = {32, 16, 1};
    __host__ __device__ static constexpr int r(int s) { return s == 0 ? 32 : s == 1 ? 16 : 1; } };
template <> struct WPlan<10>  { static constexpr int NP = 2, TPL = 32; static constexpr int R[3] = {32, 32, 1};
    __host__ __device__ static constexpr int r(int s) { return s == 0 ? 32 : s == 1 ? 32 : 1; } };

// Twiddle sources.  A source answers get<S>(i, r, k, t) for pass S: item i of the lane, leg r,
// k = position of the item inside its sub-transform, t = index into a full N-point table (the
// twiddle wanted is exp(-2 pi i t / N); the engine conjugates it for inverse transforms).
template <int N> struct TableTw {               // full table of N entries in shared memory
    const float2 *tw;
    template <int S> __device__ __forceinline__ float2 get(int, int, int, int t) const { return tw[t]; }
};

template <int LOG2N, bool INV> struct WF {
    using P = WPlan<LOG2N>;
    static constexpr int N = 1 << LOG2N;
    static constexpr int NP = P::NP;
    static constexpr int TPL = P::TPL;
    static constexpr int LPW = 32 / TPL;                  // lines per warp
    // mask of the lanes that share a line with this thread (argument `m` of the functions below)
    static __device__ __forceinline__ unsigned group_mask(int tid)
    {
        return TPL == 32 ? 0xffffffffu : (((1u << TPL) - 1u) << ((tid & 31) / TPL * TPL));
    }
    __host__ __device__ static constexpr int radix(int s) { return INV ? P::r(NP - 1 - s) : P::r(s); }
    __host__ __device__ static constexpr int ns(int s)
    {
        int n = 1;
        for (int i = 0; i < s; ++i) n *= radix(i);
        return n;
    }
    // Lines are stored skewed: position i sits at ph(i).  The shift follows the radix of the first
    // pass, whose results land R points apart per lane: with it the groups of a warp that work on
    // neighbouring lines never meet in a bank.
    static constexpr int SKEW = (LOG2N <= 7 && radix(0) == 8) ? 3 : radix(0) == 32 ? 5 : 4;
    __host__ __device__ static constexpr int ph(int i) { return i + (i >> SKEW); }
    template <int S> struct Pass {
        static constexpr int R = radix(S);
        static constexpr int NS = ns(S);
        static constexpr int ITEMS = N / R;
        static constexpr int IPL = ITEMS >= TPL ? ITEMS / TPL : 1;   // items per lane
        static constexpr bool PARTIAL = ITEMS < TPL;                 // only lanes < ITEMS work
    };

    // One pass.  in(i, r, idx) -> float2 gives the point at position idx (item i of this
    // lane, leg r); out(i, r, idx, v) receives the result for position idx.
    // PR: PRUNE_IN (first pass only: positions >= N/2 are zero and never requested),
    //     PRUNE_OUT (last pass only: positions >= N/2 are not produced).
    // tw: twiddle source (see TableTw).
    template <int S, int PR, class Tw, class In, class Out>
    static __device__ __forceinline__ void pass(int l, Tw tw, In in, Out out)
    {
        using PS = Pass<S>;
        constexpr int R = PS::R, NS = PS::NS;
        constexpr int NIN = (PR == PRUNE_IN) ? R / 2 : R;
        constexpr int NOUT = (PR == PRUNE_OUT) ? R / 2 : R;
        if (PS::PARTIAL && l >= PS::ITEMS) return;
#pragma unroll
        for (int i = 0; i < PS::IPL; ++i) {
            const int j = l + i * TPL;
            float2 x[R];
#pragma unroll
            for (int r = 0; r < NIN; ++r) x[r] = in(i, r, j + r * (N / R));
#pragma unroll
            for (int r = NIN; r < R; ++r) x[r] = make_float2(0.f, 0.f);
            if constexpr (NS > 1) {
                const int k = j & (NS - 1);
#pragma unroll
                for (int r = 1; r < NIN; ++r) {
                    const float2 w = tw.template get<S>(i, r, k, r * k * (N / (NS * R)));
                    x[r] = INV ? cmulc(x[r], w) : cmul(x[r], w);
                }
            }
            dft<R, INV, PR>(x);
            const int k = j & (NS - 1);
            const int base = (j - k) * R + k;
#pragma unroll
            for (int r = 0; r < NOUT; ++r) out(i, r, base + r * NS, x[r]);
        }
    }

    // Passes [S0, S1) line -> line, each followed by __syncwarp().  PR0 applies to pass S0
    // (PRUNE_IN is only meaningful when S0 == 0).
    template <int S0, int S1, int PR0 = PRUNE_NONE, class Tw>
    static __device__ __forceinline__ void mid(int l, unsigned m, Tw tw, float2 *line)
    {
        if constexpr (S0 < S1) {
            // loads of all items must precede the stores of any item of the same line
            using PS = Pass<S0>;
            constexpr int R = PS::R;
            float2 keep[PS::IPL][R];
            pass<S0, PR0>(l, tw,
                [&](int, int, int idx) { return line[ph(idx)]; },
                [&](int i, int r, int, float2 v) { keep[i][r] = v; });
            __syncwarp(m);
            if (!(PS::PARTIAL && l >= PS::ITEMS)) {
#pragma unroll
                for (int i = 0; i < PS::IPL; ++i) {
                    const int j = l + i * TPL;
                    const int k = j & (PS::NS - 1);
                    const int base = (j - k) * R + k;
#pragma unroll
                    for (int r = 0; r < R; ++r) line[ph(base + r * PS::NS)] = keep[i][r];
                }
            }
            __syncwarp(m);
            mid<S0 + 1, S1, PRUNE_NONE>(l, m, tw, line);
        }
    }

    // Full transform: first-pass inputs from `in`, last-pass outputs to `out`; the line is
    // scratch.  Callers must __syncwarp() before reusing the line for something else.
    // ALIAS: the first-pass inputs live in the line itself (in another format), so all of them
    // are read before the first pass writes its results.
    template <int PR, bool ALIAS = false, class Tw, class In, class Out>
    static __device__ __forceinline__ void run(int l, unsigned m, Tw tw, float2 *line, In in, Out out)
    {
        constexpr int PF = (PR == PRUNE_IN) ? PRUNE_IN : PRUNE_NONE;
        constexpr int PL = (PR == PRUNE_OUT) ? PRUNE_OUT : PRUNE_NONE;
        if constexpr (ALIAS) {
            using P0 = Pass<0>;
            float2 keep[P0::IPL][P0::R];
            pass<0, PF>(l, tw, in, [&](int i, int r, int, float2 v) { keep[i][r] = v; });
            __syncwarp(m);
            if (!(P0::PARTIAL && l >= P0::ITEMS)) {
#pragma unroll
                for (int i = 0; i < P0::IPL; ++i)
#pragma unroll
                    for (int r = 0; r < P0::R; ++r) line[ph((l + i * TPL) * P0::R + r)] = keep[i][r];
            }
        } else {
            pass<0, PF>(l, tw, in, [&](int, int, int idx, float2 v) { line[ph(idx)] = v; });
        }
        __syncwarp(m);
        mid<1, NP - 1, PRUNE_NONE>(l, m, tw, line);
        pass<NP - 1, PL>(l, tw, [&](int, int, int idx) { return line[ph(idx)]; }, out);
    }

    // Position (natural order) of output leg r of item i of lane l after the last pass.
    using LastPass = Pass<NP - 1>;
    static __device__ __forceinline__ int last_pos(int l, int i, int r) { return l + i * TPL + r * (N / LastPass::R); }

    // Register copy of the twiddles of pass S (they depend on the lane only).
    template <int S> struct Hoist {
        using PS = Pass<S>;
        float2 w[PS::IPL][PS::R];
        __device__ __forceinline__ void load(int l, const float2 *table)
        {
#pragma unroll
            for (int i = 0; i < PS::IPL; ++i) {
                const int k = (l + i * TPL) & (PS::NS - 1);
#pragma unroll
                for (int r = 1; r < PS::R; ++r) w[i][r] = table[r * k * (N / (PS::NS * PS::R))];
            }
        }
        template <int S2> __device__ __forceinline__ float2 get(int i, int r, int, int) const { return w[i][r]; }
    };

    // Full transform whose results end up in the line itself (natural order); ends with a
    // __syncwarp(), so every lane of the group may read any position afterwards.
    template <int PR, bool ALIAS = false, class Tw, class In>
    static __device__ __forceinline__ void run_to_line(int l, unsigned m, Tw tw, float2 *line, In in)
    {
        using PS = Pass<NP - 1>;
        float2 keep[PS::IPL][PS::R];
        run<PR, ALIAS>(l, m, tw, line, in, [&](int i, int r, int, float2 v) { keep[i][r] = v; });
        __syncwarp(m);
        if (!(PS::PARTIAL && l >= PS::ITEMS)) {
            constexpr int NOUT = (PR == PRUNE_OUT) ? PS::R / 2 : PS::R;
#pragma unroll
            for (int i = 0; i < PS::IPL; ++i) {
                const int j = l + i * TPL;
#pragma unroll
                for (int r = 0; r < NOUT; ++r) line[ph(j + r * (N / PS::R))] = keep[i][r];
            }
        }
        __syncwarp(m);
    }
};

// Per-pass twiddle tables in shared memory, laid out [leg][k] so that the lanes of a warp (which
// differ in k) read consecutive entries: no bank conflicts, unlike a shared N-point table.
template <int LOG2N, bool INV> struct PassTw {
    using F = WF<LOG2N, INV>;
    const float2 *base;
    __host__ __device__ static constexpr int size(int s) { return s == 0 ? 0 : (F::radix(s) - 1) * F::ns(s); }
    __host__ __device__ static constexpr int offset(int s)
    {
        int o = 0;
        for (int i = 0; i < s; ++i) o += size(i);
        return o;
    }
    static constexpr int TOTAL = offset(F::NP);
    // gtw: global table of gtw_n >= N points; all nthr threads take part; caller synchronises
    static __device__ __forceinline__ void build(float2 *dst, const float2 *gtw, int gtw_n, int tid, int nthr)
    {
        constexpr int N = 1 << LOG2N;
        const int step = gtw_n >> LOG2N;
        for (int s = 1; s < F::NP; ++s) {
            const int ns = F::ns(s), rad = F::radix(s), off = offset(s);
            for (int e = tid; e < (rad - 1) * ns; e += nthr) {
                const int r = e / ns + 1, k = e % ns;
                HN_G(gtw + r * k * (N / (ns * rad)) * step, 8);
                dst[off + e] = gtw[r * k * (N / (ns * rad)) * step];
            }
        }
    }
    template <int S> __device__ __forceinline__ float2 get(int, int r, int k, int) const
    {
        return base[offset(S) + (r - 1) * F::ns(S) + k];
    }
};

}  // namespace hn
