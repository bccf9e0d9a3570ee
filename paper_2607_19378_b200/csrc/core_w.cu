// Fused spectral core along a strided axis, warp-engine version.
//
// For a tile of adjacent bins the CTA loads the k*v lines and the filter lines
// (coalesced rows, transposed into shared-memory lines), and each group of lanes
// then owns one line: forward transform of the filter line into registers,
// forward transform of the k*v line into registers, spectral product (Eq. 12 of
// the paper), and the inverse transform started from those registers.  Only the
// cropped half of the inverse is produced and written back in place.
#include "common.cuh"
#include "plane_util.cuh"

namespace hn {

// threads per CTA.  For 1024-point lines (one CTA of 8 groups per SM) both 12 groups per CTA and three CTAs of
// 4 groups were measured slower: tiles that are not 64 bytes wide per row cost more than the extra warps give.
__host__ __device__ constexpr int core_threads(int) { return 256; }

__device__ __forceinline__ void cp_async8(void *smem_dst, const void *gmem_src)
{
    const unsigned d = (unsigned)__cvta_generic_to_shared(smem_dst);
    HN_G(gmem_src, 8);
    asm volatile("cp.async.ca.shared.global [%0], [%1], 8;\n" ::"r"(d), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async8_s(unsigned smem_addr, const void *gmem_src)
{
    HN_G(gmem_src, 8);
    asm volatile("cp.async.ca.shared.global [%0], [%1], 8;\n" ::"r"(smem_addr), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory"); }

// Line stride.  Tile copies and the final stores walk the lines with one lane per line (x) and
// row (pos): with 16 or more lines per tile a half warp touches 16 lines at one row and any odd stride
// separates them; with 8 lines it touches 8 lines at two neighbouring rows, which a stride of
// 2 mod 16 separates.
template <int LOG2P> __host__ __device__ constexpr int core_ls()
{
    using F = WF<LOG2P, false>;
    constexpr int N = 1 << LOG2P, TX = core_threads(LOG2P) / F::TPL;
    if (TX >= 16) return line_stride(N);
    int n = (F::ph(N - 1) > WF<LOG2P, true>::ph(N - 1) ? F::ph(N - 1) : WF<LOG2P, true>::ph(N - 1)) + 1;
    while (n % 16 != 2) ++n;
    return n;
}

// FULL (circular mode: n_in == n_out == N): the k*v lines have no zero half and every output is kept.
template <int LOG2P, bool FULL>
__global__ void __launch_bounds__(core_threads(LOG2P), (LOG2P >= 10 ? 1 : 2)) axis_core_w_kernel(AxisArgs p)
{
    constexpr int kCoreThreads = core_threads(LOG2P);
    using F = WF<LOG2P, false>;
    using FI = WF<LOG2P, true>;
    constexpr int N = 1 << LOG2P, TPL = F::TPL, NP = F::NP;
    constexpr int TX = kCoreThreads / TPL;                 // lines per tile
    constexpr int LS = core_ls<LOG2P>();
    using PL = typename F::template Pass<NP - 1>;          // last forward pass == first inverse pass
    extern __shared__ float2 smem[];
    float2 *bu = smem;
    float2 *bh = smem + TX * LS;
    float2 *twt = smem + 2 * TX * LS;
    const int tid = threadIdx.x, l = tid % TPL, gid = tid / TPL;
    const unsigned m = F::group_mask(tid);
    float2 *uline = bu + gid * LS;
    float2 *hline = bh + gid * LS;
    for (int t = tid; t < N; t += kCoreThreads) { HN_G(p.gtw + t * (p.gtw_n / N), 8); twt[t] = p.gtw[t * (p.gtw_n / N)]; }
    __syncthreads();
    // twiddles: registers when both passes are equal (they depend on the lane only), else
    // per-pass tables
    PlaneTw<LOG2P, false> tw;
    tw.init(l, twt, twt + N, tid, kCoreThreads);
    PlaneTw<LOG2P, true> twi;
    twi.init(l, twt, twt + N + PlaneTw<LOG2P, false>::TABLE, tid, kCoreThreads);
    __syncthreads();
    const long long tpo = (p.nc + TX - 1) / TX;
    const long long tiles = p.n_outer * tpo;
    // Tile loads are asynchronous copies (one complex bin per thread and row) straight into the
    // lines; the filter lines of the next tile are fetched while this tile's k*v lines are
    // transformed, and the next k*v lines while the next filter lines are transformed.
    constexpr int RPS = kCoreThreads / TX;                 // rows per step
    const int x = tid % TX, r0 = tid / TX;
    // Row pos of the padded line holds filter row (pos + h_shift) mod N: rows [h_shift, h_n_in) sit at
    // positions [0, h_n_in - h_shift), rows [0, h_shift) at [N - h_shift, N), the gap is zero.  Each
    // thread walks its positions with running pointers (no wrap arithmetic per copy).
    const unsigned bh_x = (unsigned)__cvta_generic_to_shared(bh + x * LS);
    const unsigned bu_x = (unsigned)__cvta_generic_to_shared(bu + x * LS);
    auto issue_h = [&](long long t) {
        const long long o = t / tpo;
        const int c0 = (int)(t % tpo) * TX;
        const long long oh = p.h_mod ? (o + p.h_off) % p.h_mod : o;
        const float2 *hs = p.h + oh * p.h_outer + c0 + x;
        const bool inside = c0 + x < p.nc;
        const int head = p.h_n_in - p.h_shift;             // positions [0, head) <- rows [h_shift, h_n_in)
        const int tail0 = N - p.h_shift;                   // positions [tail0, N) <- rows [0, h_shift)
        const long long step = (long long)RPS * p.nc;
        if (inside) {
            const float2 *src = hs + (long long)(p.h_shift + r0) * p.nc;
#pragma unroll 4
            for (int pos = r0; pos < head; pos += RPS, src += step)
                cp_async8_s(bh_x + 8u * (unsigned)F::ph(pos), src);
            int pos = tail0 + ((r0 - tail0) & (RPS - 1));   // first position >= tail0 owned by this thread
            src = hs + (long long)(pos - tail0) * p.nc;
#pragma unroll 4
            for (; pos < N; pos += RPS, src += step)
                cp_async8_s(bh_x + 8u * (unsigned)F::ph(pos), src);
            for (int z = head + ((r0 - head) & (RPS - 1)); z < tail0; z += RPS)
                bh[x * LS + F::ph(z)] = make_float2(0.f, 0.f);
        } else {
            for (int pos = r0; pos < N; pos += RPS) bh[x * LS + F::ph(pos)] = make_float2(0.f, 0.f);
        }
    };
    auto issue_u = [&](long long t) {
        const long long o = t / tpo;
        const int c0 = (int)(t % tpo) * TX;
        const float2 *us = p.in + o * p.in_outer + c0 + x;
        const bool inside = c0 + x < p.nc;
        const int nin = inside ? p.n_in : 0;
        const long long step = (long long)RPS * p.nc;
        const float2 *src = us + (long long)r0 * p.nc;
        int pos = r0;
#pragma unroll 4
        for (; pos < nin; pos += RPS, src += step) cp_async8_s(bu_x + 8u * (unsigned)F::ph(pos), src);
        for (; pos < (FULL ? N : N / 2); pos += RPS) bu[x * LS + F::ph(pos)] = make_float2(0.f, 0.f);
    };
    long long t = blockIdx.x;
    if (t < tiles) { issue_h(t); }
    cp_async_commit();
    if (t < tiles) { issue_u(t); }
    cp_async_commit();
    while (t < tiles) {
        const long long tn = t + gridDim.x;
        using PL2 = PL;
        constexpr bool HREG = PL2::IPL * PL2::R <= 16;
        float2 H[HREG ? PL2::IPL : 1][HREG ? PL2::R : 1];
        cp_async_wait<1>();                                // filter lines of this tile have landed
        __syncthreads();
        if constexpr (HREG) {
            F::template mid<0, NP - 1, PRUNE_NONE>(l, m, tw, hline);
            F::template pass<NP - 1, PRUNE_NONE>(l, tw,
                [&](int, int, int idx) { return hline[F::ph(idx)]; },
                [&](int i, int r, int, float2 v) { H[i][r] = make_float2(v.x * p.scale, v.y * (p.h_conj ? -p.scale : p.scale)); });
            __syncthreads();                               // filter lines are free again
            if (tn < tiles) issue_h(tn);
            cp_async_commit();
            cp_async_wait<1>();                            // k*v lines of this tile have landed
        } else {
            F::template mid<0, NP, PRUNE_NONE>(l, m, tw, hline);   // spectrum stays in the line
            cp_async_wait<0>();
        }
        __syncthreads();
        {
            F::template mid<0, NP - 1, FULL ? PRUNE_NONE : PRUNE_IN>(l, m, tw, uline);
            float2 Y[PL::IPL][PL::R];
            F::template pass<NP - 1, PRUNE_NONE>(l, tw,
                [&](int, int, int idx) { return uline[F::ph(idx)]; },
                [&](int i, int r, int idx, float2 v) {
                    if constexpr (HREG) Y[i][r] = cmul(v, H[i][r]);
                    else {
                        const float2 hh = hline[F::ph(idx)];
                        Y[i][r] = cmul(v, make_float2(hh.x * p.scale, hh.y * (p.h_conj ? -p.scale : p.scale)));
                    }
                });
            __syncwarp(m);
            FI::template pass<0, PRUNE_NONE>(l, twi,
                [&](int i, int r, int) { return Y[i][r]; },
                [&](int, int, int idx, float2 v) { uline[FI::ph(idx)] = v; });
            __syncwarp(m);
            FI::template mid<1, NP - 1, PRUNE_NONE>(l, m, twi, uline);
            using PE = typename FI::template Pass<NP - 1>;
            float2 keep[PE::IPL][PE::R];
            FI::template pass<NP - 1, FULL ? PRUNE_NONE : PRUNE_OUT>(l, twi,
                [&](int, int, int idx) { return uline[FI::ph(idx)]; },
                [&](int i, int r, int, float2 v) { keep[i][r] = v; });
            __syncwarp(m);
            if (!(PE::PARTIAL && l >= PE::ITEMS)) {
#pragma unroll
                for (int i = 0; i < PE::IPL; ++i)
#pragma unroll
                    for (int r = 0; r < (FULL ? PE::R : PE::R / 2); ++r)
                        uline[FI::ph(l + i * TPL + r * (N / PE::R))] = keep[i][r];
            }
        }
        __syncthreads();
        if constexpr (!HREG) {
            if (tn < tiles) issue_h(tn);
            cp_async_commit();
        }
        {
            const long long o = t / tpo;
            const int c0 = (int)(t % tpo) * TX;
            float2 *dst = p.out + o * p.out_outer + c0 + x + (long long)r0 * p.nc;
            const long long step = (long long)RPS * p.nc;
            if (c0 + x < p.nc)
                for (int pos = r0; pos < p.n_out; pos += RPS, dst += step) { HN_G(dst, 8); *dst = bu[x * LS + FI::ph(pos)]; }
        }
        __syncthreads();
        if (tn < tiles) issue_u(tn);
        cp_async_commit();
        t = tn;
    }
    cp_async_wait<0>();
}

template <int LOG2P, bool FULL> static int launch_core_w_t(const AxisArgs &a, cudaStream_t st)
{
    using F = WF<LOG2P, false>;
    constexpr int kCoreThreads = core_threads(LOG2P);
    constexpr int N = 1 << LOG2P, TX = kCoreThreads / F::TPL;
    const size_t sm = sizeof(float2) * ((size_t)2 * TX * core_ls<LOG2P>() + N + PlaneTw<LOG2P, false>::TABLE + PlaneTw<LOG2P, true>::TABLE);
    static int sms = 0;
    if (!sms) {
        int dev = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (sms <= 0) sms = 148;
    }
    static DevOnce attr;
    if (attr.first()) cudaFuncSetAttribute(axis_core_w_kernel<LOG2P, FULL>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
    const long long tiles = a.n_outer * ((a.nc + TX - 1) / TX);
    const long long res = (long long)sms * 2;
    const int grid = (int)(tiles < res ? tiles : res);
    if (grid <= 0) return 0;
    axis_core_w_kernel<LOG2P, FULL><<<grid, kCoreThreads, sm, st>>>(a);
    return 1;
}

// ---- one transform along a strided axis (the middle axis of 3-D grids on the general path) ------------------------
// Same tiles and lane groups as the core above, one transform per line: forward (PRUNE: the upper half of the padded
// input is zero) from n_in entries, placed at (m - shift) mod N, to n_out <= N bins; or inverse from n_in <= N bins to
// n_out entries (PRUNE: only the lower half is produced, n_out <= N/2).  Lines are read from `in` and written to `out`
// (different buffers, their own outer strides).
template <int LOG2P, bool INV, bool PRUNE>
__global__ void __launch_bounds__(core_threads(LOG2P), (LOG2P >= 10 ? 1 : 2)) axis_w_kernel(AxisArgs p)
{
    constexpr int kCoreThreads = core_threads(LOG2P);
    using F = WF<LOG2P, INV>;
    constexpr int N = 1 << LOG2P, TPL = F::TPL;
    constexpr int TX = kCoreThreads / TPL;
    constexpr int LS = core_ls<LOG2P>();
    extern __shared__ float2 smem[];
    float2 *bu = smem;
    float2 *twt = smem + TX * LS;
    const int tid = threadIdx.x, l = tid % TPL, gid = tid / TPL;
    const unsigned m = F::group_mask(tid);
    float2 *line = bu + gid * LS;
    for (int t = tid; t < N; t += kCoreThreads) { HN_G(p.gtw + t * (p.gtw_n / N), 8); twt[t] = p.gtw[t * (p.gtw_n / N)]; }
    __syncthreads();
    PlaneTw<LOG2P, INV> tw;
    tw.init(l, twt, twt + N, tid, kCoreThreads);
    __syncthreads();
    const long long tpo = (p.nc + TX - 1) / TX;
    const long long tiles = p.n_outer * tpo;
    constexpr int RPS = kCoreThreads / TX;                 // rows per step
    const int x = tid % TX, r0 = tid / TX;
    const unsigned bu_x = (unsigned)__cvta_generic_to_shared(bu + x * LS);
    constexpr int NFILL = (!INV && PRUNE) ? N / 2 : N;     // positions the first pass reads
    for (long long t = blockIdx.x; t < tiles; t += gridDim.x) {
        const long long o = t / tpo;
        const int c0 = (int)(t % tpo) * TX;
        const bool inside = c0 + x < p.nc;
        const float2 *us = p.in + o * p.in_outer + c0 + x;
        const long long step = (long long)RPS * p.nc;
        if (inside) {
            // position pos holds entry (pos + shift) mod N: entries [shift, n_in) sit at [0, n_in - shift), entries
            // [0, shift) at [N - shift, N), the gap is zero
            const int head = p.n_in - p.shift, tail0 = N - p.shift;
            const float2 *src = us + (long long)(p.shift + r0) * p.nc;
            for (int pos = r0; pos < head && pos < NFILL; pos += RPS, src += step) cp_async8_s(bu_x + 8u * (unsigned)F::ph(pos), src);
            if (p.shift) {
                int pos = tail0 + ((r0 - tail0) & (RPS - 1));
                src = us + (long long)(pos - tail0) * p.nc;
                for (; pos < NFILL; pos += RPS, src += step) cp_async8_s(bu_x + 8u * (unsigned)F::ph(pos), src);
            }
            const int z1 = p.shift ? tail0 : N;
            for (int z = (head > 0 ? head : 0) + ((r0 - (head > 0 ? head : 0)) & (RPS - 1)); z < z1 && z < NFILL; z += RPS)
                bu[x * LS + F::ph(z)] = make_float2(0.f, 0.f);
        } else {
            for (int pos = r0; pos < NFILL; pos += RPS) bu[x * LS + F::ph(pos)] = make_float2(0.f, 0.f);
        }
        cp_async_commit();
        cp_async_wait<0>();
        __syncthreads();
        constexpr int PR = PRUNE ? (INV ? PRUNE_OUT : PRUNE_IN) : PRUNE_NONE;
        F::template run_to_line<PR, true>(l, m, tw, line, [&](int, int, int idx) { return line[F::ph(idx)]; });
        __syncthreads();
        if (inside) {
            float2 *dst = p.out + o * p.out_outer + c0 + x + (long long)r0 * p.nc;
            for (int pos = r0; pos < p.n_out; pos += RPS, dst += step) { HN_G(dst, 8); *dst = bu[x * LS + F::ph(pos)]; }
        }
        __syncthreads();
    }
}

template <int LOG2P, bool INV, bool PRUNE> static int launch_axis_w_t(const AxisArgs &a, cudaStream_t st)
{
    using F = WF<LOG2P, INV>;
    constexpr int kCoreThreads = core_threads(LOG2P);
    constexpr int N = 1 << LOG2P, TX = kCoreThreads / F::TPL;
    const size_t sm = sizeof(float2) * ((size_t)TX * core_ls<LOG2P>() + N + PlaneTw<LOG2P, INV>::TABLE);
    static int sms = 0;
    if (!sms) {
        int dev = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (sms <= 0) sms = 148;
    }
    static DevOnce attr;
    if (attr.first()) cudaFuncSetAttribute(axis_w_kernel<LOG2P, INV, PRUNE>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
    const long long tiles = a.n_outer * ((a.nc + TX - 1) / TX);
    const long long res = (long long)sms * (LOG2P >= 10 ? 1 : 4);
    const int grid = (int)(tiles < res ? tiles : res);
    if (grid <= 0) return 0;
    axis_w_kernel<LOG2P, INV, PRUNE><<<grid, kCoreThreads, sm, st>>>(a);
    return 1;
}

// forward: a.prune_in selects the pruned first pass; inverse: a.full keeps every output, else the lower half
int launch_axis_w(const AxisArgs &a, bool inverse, cudaStream_t st)
{
    const int n = 1 << a.log2p;
    if (a.in == a.out) return -1;
    if (!inverse && (a.n_in > (a.prune_in ? n / 2 : n) || a.n_out > n || a.shift < 0 || a.shift >= n || (a.prune_in && a.shift))) return -1;
    if (inverse && (a.n_in > n || a.shift || a.n_out > (a.full ? n : n / 2))) return -1;
#define HN_AXW(L)                                                                                       \
    case L:                                                                                             \
        if (!inverse) return a.prune_in ? launch_axis_w_t<L, false, true>(a, st) : launch_axis_w_t<L, false, false>(a, st); \
        return a.full ? launch_axis_w_t<L, true, false>(a, st) : launch_axis_w_t<L, true, true>(a, st);
    switch (a.log2p) {
        HN_AXW(6) HN_AXW(7) HN_AXW(8) HN_AXW(9) HN_AXW(10)
    default: return -1;
    }
#undef HN_AXW
}

bool core_w_supported(int log2p) { return log2p >= 6 && log2p <= 10; }

int launch_core_w(const AxisArgs &a, cudaStream_t st)
{
    switch (a.log2p) {
    case 6: return a.full ? launch_core_w_t<6, true>(a, st) : launch_core_w_t<6, false>(a, st);
    case 7: return a.full ? launch_core_w_t<7, true>(a, st) : launch_core_w_t<7, false>(a, st);
    case 8: return a.full ? launch_core_w_t<8, true>(a, st) : launch_core_w_t<8, false>(a, st);
    case 9: return a.full ? launch_core_w_t<9, true>(a, st) : launch_core_w_t<9, false>(a, st);
    case 10: return a.full ? launch_core_w_t<10, true>(a, st) : launch_core_w_t<10, false>(a, st);
    default: return -1;
    }
}

}  // namespace hn
