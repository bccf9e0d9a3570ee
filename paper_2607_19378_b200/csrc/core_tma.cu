// Fused spectral core along a strided axis for 256- and 1024-point lines, tiles moved by TMA.
//
// Same arithmetic as core_w.cu (forward transform of the filter lines, forward transform of the
// k*v lines, spectral product of Eq. 12 of the paper, inverse, cropped half written back in
// place), but the tiles -- 8 adjacent bins by all rows of the axis -- travel as tensor copies:
//
//   cp.async.bulk.tensor loads   filter tile (boxes of up to 256 rows; the wrapped placement of the
//                                taps is two row ranges) and k*v tile (one box; rows past the data
//                                and bins past the end come back as zeros)
//   cp.async.bulk.tensor store   the cropped result tile
//
// One elected thread issues them; nobody computes addresses or waits per element.  The boxes land
// row-major (one 64-byte row per axis position; the code also covers 128-byte rows) with the matching swizzle, which
// spreads the rows a group of lanes reads at once over the banks.  A tile buffer is free again as soon as the first pass
// has read it, so the next tile's copy runs under the rest of this tile's arithmetic.
//
// Every wait on a copy is bounded: if a barrier does not complete, the CTA records it in the
// status word, waits (bounded again) for what is still in flight and returns.
#include <cuda.h>
#include <cstdint>
#include "common.cuh"
#include "plane_util.cuh"
#include "core_tma.cuh"
#include "tma_util.cuh"

namespace hn {

// Threads per CTA: 256-point lines run as 4 CTAs of 128 threads per SM (8 lines per tile), 1024-point lines as one
// CTA of 256 threads (8 lines per tile).  A CTA synchronises at two barriers per tile; more, smaller CTAs per SM
// keep the schedulers busy while one of them waits.
template <int LOG2P> struct TmaCta {
    static constexpr int THREADS = LOG2P >= 10 ? 256 : 128;
    static constexpr int PER_SM = LOG2P >= 10 ? 1 : 4;
};

// Geometry of a tile for LOG2P-point lines: one line per group of TPL lanes, so TX = THREADS / TPL bins
// per tile and TX * 8 bytes per tile row (64 here: the swizzle span of the tensor maps).  A box holds at
// most 256 rows.
template <int LOG2P> struct TmaGeo {
    using F = WF<LOG2P, false>;
    static constexpr int N = 1 << LOG2P, HALF = N / 2;
    static constexpr int THREADS = TmaCta<LOG2P>::THREADS;
    static constexpr int TX = THREADS / F::TPL;
    static constexpr unsigned ROWB = TX * 8;
    static constexpr int BOXR = HALF < 256 ? HALF : 256;             // rows per box
    static constexpr int NB = HALF / BOXR;                           // boxes per half line
    static constexpr unsigned BOXB = BOXR * ROWB;
    static constexpr unsigned HALFB = HALF * ROWB;
    // 16-lane groups (two lines per warp): the lanes of a half warp belong to both lines (see the kernel), whose
    // strides are therefore 8 mod 16 entries, i.e. half a bank row apart
    static constexpr int LS = F::TPL == 16 ? plane_ls(N) : ((F::ph(N - 1) + 1 + 15) / 16 * 16 + 2);
    static_assert(ROWB == 128 || ROWB == 64, "tile rows match a swizzle span");
    // shared memory: tile buffers first (1024-byte aligned, as the swizzle pattern repeats every 1024 bytes)
    static constexpr size_t TH = 0;                                  // filter tile, N rows
    static constexpr size_t TU = TH + 2 * HALFB;                     // k*v tile, N/2 rows
    static constexpr size_t TO = TU + HALFB;                         // result tile, N/2 rows
    static constexpr size_t LINES = TO + HALFB;                      // one skewed line per group
    static constexpr size_t TW = LINES + sizeof(float2) * TX * LS;
    static constexpr size_t BARS = TW + sizeof(float2) * N;
    static constexpr size_t TOTAL = BARS + 2 * sizeof(uint64_t) + 1024;    // + room to align the start
};

struct CoreTmaParams {
    long long n_outer;
    int tiles_per_outer;      // ceil(nc / TX)
    int h_shift;              // filter row (pos + h_shift) mod N sits at position pos
    long long h_mod, h_off;   // filter outer index = h_mod ? (o + h_off) % h_mod : o
    float scale;
    float scale_im;           // scale, or -scale where the product takes the conjugate of the filter spectrum
    const float2 *gtw;
    int gtw_n;
    int *status;              // device word: 0 ok, else which wait gave up
};

template <int LOG2P>
__global__ void __launch_bounds__(TmaCta<LOG2P>::THREADS, TmaCta<LOG2P>::PER_SM)
axis_core_tma_kernel(const __grid_constant__ CUtensorMap map_u, const __grid_constant__ CUtensorMap map_h, CoreTmaParams p)
{
    using G = TmaGeo<LOG2P>;
    using F = WF<LOG2P, false>;
    using FI = WF<LOG2P, true>;
    constexpr int N = G::N, TPL = F::TPL, NP = F::NP, kTmaThreads = G::THREADS;
    static_assert(NP == 2 && F::radix(0) == F::radix(1), "two equal passes: one register set of twiddles serves both directions");
    using PL = typename F::template Pass<NP - 1>;
    using P0 = typename F::template Pass<0>;
    static_assert(P0::IPL == 1 && PL::IPL == 1, "one item per lane and pass");
    constexpr int RSTEP = (N / P0::R) * (int)G::ROWB / 8;            // float2 between legs r and r+1 of a lane in a tile
    extern __shared__ __align__(1024) unsigned char smem_dyn[];
    // the swizzle pattern is a function of the shared-memory address: start on a 1024-byte boundary
    unsigned char *smem_raw = smem_dyn + ((1024u - (smem_u32(smem_dyn) & 1023u)) & 1023u);
    unsigned char *th = smem_raw + G::TH;
    unsigned char *tu = smem_raw + G::TU;
    unsigned char *to = smem_raw + G::TO;
    float2 *lines = reinterpret_cast<float2 *>(smem_raw + G::LINES);
    float2 *twt = reinterpret_cast<float2 *>(smem_raw + G::TW);
    uint64_t *bar_h = reinterpret_cast<uint64_t *>(smem_raw + G::BARS);
    uint64_t *bar_u = bar_h + 1;
    // Lanes of a warp: with one line per warp (32 lanes per line) lane = position.  With two lines per warp the
    // two are interleaved in blocks of 8 lanes (lanes 0-7 and 16-23 work on the first line, 8-15 and 24-31 on the
    // second): an 8-byte shared-memory access is served per half warp, and a half warp then reads 8 rows of BOTH
    // bins of a 16-byte tile chunk, 16 distinct 8-byte slots, instead of 16 rows of one bin, which share 8 slots.
    const int tid = threadIdx.x;
    const int l = TPL == 16 ? ((tid & 7) | ((tid >> 1) & 8)) : tid % TPL;
    const int gid = TPL == 16 ? ((tid >> 5) * 2 + ((tid >> 3) & 1)) : tid / TPL;
    const unsigned m = TPL == 16 ? (0x00ff00ffu << (tid & 8)) : F::group_mask(tid);
    float2 *line = lines + gid * G::LS;
    for (int t = tid; t < N; t += kTmaThreads) { HN_G(p.gtw + t * (p.gtw_n / N), 8); twt[t] = p.gtw[t * (p.gtw_n / N)]; }
    if (tid == 0) {
        mbar_init(bar_h, 1);
        mbar_init(bar_u, 1);
        fence_mbar_init();
    }
    __syncthreads();
    // two equal passes: the twiddles depend on the lane only and live in registers; the inverse uses the
    // same values conjugated, so one set serves both directions
    PlaneTw<LOG2P, false> tw;
    static_assert(PlaneTw<LOG2P, false>::HOIST, "register twiddles");
    tw.init(l, twt, twt, tid, kTmaThreads);
    // Row z = l + TPL*r of bin `gid` inside a swizzled tile.  A row is ROWB bytes; the 16-byte chunk index
    // of an address is XORed with address bits 7 and up (3 bits for the 128-byte swizzle, 2 for the 64-byte
    // one), i.e. with a function of z that TPL*r does not change: every leg r is the same per-lane offset
    // plus a constant.
    constexpr unsigned ZSH = G::ROWB == 128 ? 0 : 1, ZMASK = G::ROWB == 128 ? 7u : 3u;
    const unsigned tile_off = (unsigned)l * G::ROWB
                            + ((((unsigned)gid >> 1) ^ (((unsigned)l >> ZSH) & ZMASK)) << 4) + ((unsigned)gid & 1u) * 8u;
    const long long tiles = p.n_outer * p.tiles_per_outer;
    auto issue_h = [&](long long t) {                  // one thread
        const long long o = t / p.tiles_per_outer;
        const int x = (int)(t % p.tiles_per_outer) * G::TX * 2;          // in floats
        const long long oh = p.h_mod ? (o + p.h_off) % p.h_mod : o;
        mbar_expect_tx(bar_h, 2 * G::HALFB);
#pragma unroll
        for (int b = 0; b < G::NB; ++b) {
            // positions [0, N/2) hold filter rows from h_shift on, positions [N/2, N) the rows before it
            tma_load_3d(th + b * G::BOXB, &map_h, bar_h, x, p.h_shift + b * G::BOXR, (int)oh);
            tma_load_3d(th + G::HALFB + b * G::BOXB, &map_h, bar_h, x, p.h_shift - G::HALF + b * G::BOXR, (int)oh);
        }
    };
    auto issue_u = [&](long long t) {
        const long long o = t / p.tiles_per_outer;
        const int x = (int)(t % p.tiles_per_outer) * G::TX * 2;
        mbar_expect_tx(bar_u, G::HALFB);
#pragma unroll
        for (int b = 0; b < G::NB; ++b) tma_load_3d(tu + b * G::BOXB, &map_u, bar_u, x, b * G::BOXR, (int)o);
    };
    auto store_tile = [&](long long t) {               // one thread
        const long long o = t / p.tiles_per_outer;
        const int x = (int)(t % p.tiles_per_outer) * G::TX * 2;
#pragma unroll
        for (int b = 0; b < G::NB; ++b) tma_store_3d(&map_u, to + b * G::BOXB, x, b * G::BOXR, (int)o);
        tma_commit();
    };
    long long t = blockIdx.x, tprev = 0;
    bool have_prev = false;
    if (tid == 0 && t < tiles) { issue_h(t); issue_u(t); }
    unsigned phase = 0;
    int failed = 0;
    for (; t < tiles; t += gridDim.x, phase ^= 1u) {
        const long long tn = t + gridDim.x;
        float2 H[PL::R];
        // ---- filter lines: tile -> registers ------------------------------------------------------
        if (!mbar_wait(bar_h, phase)) failed = 1;
        {
            const float2 *src = reinterpret_cast<const float2 *>(th + tile_off);
            F::template pass<0, PRUNE_NONE>(l, tw,
                [&](int, int r, int) { return src[r * RSTEP]; },
                [&](int, int, int idx, float2 v) { line[F::ph(idx)] = v; });
        }
        if (__syncthreads_or(failed)) break;           // the filter tile buffer is free again; the previous result tile is complete
        if (tid == 0) {
            if (have_prev) store_tile(tprev);          // (its writers fenced before this barrier)
            if (tn < tiles) issue_h(tn);
        }
        F::template pass<NP - 1, PRUNE_NONE>(l, tw,
            [&](int, int, int idx) { return line[F::ph(idx)]; },
            [&](int, int r, int, float2 v) { H[r] = make_float2(v.x * p.scale, v.y * p.scale_im); });
        __syncwarp(m);
        // ---- k*v lines: tile -> spectrum, product, inverse ----------------------------------------
        if (!mbar_wait(bar_u, phase)) failed = 2;
        {
            const float2 *src = reinterpret_cast<const float2 *>(tu + tile_off);
            F::template pass<0, PRUNE_IN>(l, tw,
                [&](int, int r, int) { return src[r * RSTEP]; },
                [&](int, int, int idx, float2 v) { line[F::ph(idx)] = v; });
        }
        if (tid == 0) tma_wait_read0();                // the previous result tile has left its buffer
        if (__syncthreads_or(failed)) break;           // the k*v tile buffer is free again
        if (tid == 0 && tn < tiles) issue_u(tn);
        float2 Y[PL::R];
        F::template pass<NP - 1, PRUNE_NONE>(l, tw,
            [&](int, int, int idx) { return line[F::ph(idx)]; },
            [&](int, int r, int, float2 v) { Y[r] = cmul(v, H[r]); });
        __syncwarp(m);
        FI::template pass<0, PRUNE_NONE>(l, tw,
            [&](int, int r, int) { return Y[r]; },
            [&](int, int, int idx, float2 v) { line[FI::ph(idx)] = v; });
        __syncwarp(m);
        {
            float2 *dst = reinterpret_cast<float2 *>(to + tile_off);
            FI::template pass<NP - 1, PRUNE_OUT>(l, tw,
                [&](int, int, int idx) { return line[FI::ph(idx)]; },
                [&](int, int r, int, float2 v) { dst[r * RSTEP] = v; });
        }
        __syncwarp(m);
        fence_async_smem();                            // generic-proxy writes visible to the copy engine
        // the tile is sent after the next barrier every thread passes (the first one of the next tile, or the
        // one after the loop): no barrier of its own
        tprev = t;
        have_prev = true;
    }
    if (t >= tiles) {
        __syncthreads();
        if (tid == 0 && have_prev) store_tile(tprev);
    }
    if (t < tiles) {
        // a wait gave up: say so, then give copies that may still be in flight a bounded time to land
        if (failed) atomicExch(p.status, failed);
        mbar_wait(bar_h, phase);
        mbar_wait(bar_u, phase);
    }
    if (tid == 0) tma_wait_all0();
}

// ---- host side -------------------------------------------------------------------------------------------

// [outer][rows][nc] complex fp32, seen as fp32 with 2*nc entries per row; box = one tile row of 2*TX floats
// by up to 256 rows, swizzled over the row's 64 or 128 bytes
static bool make_map(CUtensorMap *map, const float2 *base, long long outer, int rows, int nc, long long outer_stride_elems,
                     int tx, int box_rows)
{
    const unsigned long long dims[3] = {2ull * nc, (unsigned long long)rows, (unsigned long long)outer};
    const unsigned long long strides[2] = {(unsigned long long)nc * 8, (unsigned long long)outer_stride_elems * 8};
    const unsigned box[3] = {(unsigned)tx * 2, (unsigned)box_rows, 1};
    return tma_encode_3d(map, base, /*bf16=*/false, dims, strides, box, tx * 8);
}

static bool tma_log2p_ok(int log2p) { return log2p == 8 || log2p == 10; }

bool core_tma_supported(const AxisArgs &a)
{
    if (!tma_log2p_ok(a.log2p)) return false;
    const int n = 1 << a.log2p;
    return a.in == a.out && a.in_outer == a.out_outer && a.n_in == a.n_out && a.n_in >= 1 && a.n_in <= n / 2 &&
           a.h_n_in >= 1 && a.h_n_in <= n && a.shift == 0 && a.h_shift >= 0 && a.h_shift < n && (a.nc % 2) == 0 &&
           a.n_outer < (1ll << 31) && tma_available();
}

bool core_tma_make(CoreTmaMaps *m, const AxisArgs &a, long long max_outer, long long h_outer_count)
{
    m->valid = false;
    if (!core_tma_supported(a)) return false;
    static_assert(sizeof(m->u) >= sizeof(CUtensorMap) && sizeof(m->h) >= sizeof(CUtensorMap), "room for a tensor map");
    const int tx = a.log2p == 8 ? TmaGeo<8>::TX : TmaGeo<10>::TX;
    const int br = a.log2p == 8 ? TmaGeo<8>::BOXR : TmaGeo<10>::BOXR;
    if (!make_map(reinterpret_cast<CUtensorMap *>(m->u), a.in, max_outer, a.n_in, a.nc, a.in_outer, tx, br)) return false;
    if (!make_map(reinterpret_cast<CUtensorMap *>(m->h), a.h, h_outer_count, a.h_n_in, a.nc, a.h_outer, tx, br)) return false;
    m->in = a.in; m->h_base = a.h; m->nc = a.nc; m->n_in = a.n_in; m->h_n_in = a.h_n_in; m->log2p = a.log2p;
    m->in_outer = a.in_outer; m->h_outer = a.h_outer; m->max_outer = max_outer; m->h_outer_count = h_outer_count;
    m->valid = true;
    return true;
}

template <int LOG2P> static int launch_core_tma_t(const CoreTmaParams &p0, const CoreTmaMaps &m, int nc, cudaStream_t st)
{
    using G = TmaGeo<LOG2P>;
    CoreTmaParams p = p0;
    p.tiles_per_outer = (nc + G::TX - 1) / G::TX;
    static int sms = 0;
    if (!sms) {
        int dev = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (sms <= 0) sms = 148;
    }
    static DevOnce attr;
    if (attr.first())
        cudaFuncSetAttribute(axis_core_tma_kernel<LOG2P>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)G::TOTAL);
    const long long tiles = p.n_outer * p.tiles_per_outer;
    const long long res = (long long)sms * TmaCta<LOG2P>::PER_SM;    // resident CTAs
    const int grid = (int)(tiles < res ? tiles : res);
    if (grid <= 0) return 0;
    axis_core_tma_kernel<LOG2P><<<grid, G::THREADS, G::TOTAL, st>>>(
        *reinterpret_cast<const CUtensorMap *>(m.u), *reinterpret_cast<const CUtensorMap *>(m.h), p);
    return 1;
}

int launch_core_tma(const AxisArgs &a, const CoreTmaMaps &m, int *status, cudaStream_t st)
{
    // the maps describe fixed buffers: refuse anything else
    if (!m.valid || a.log2p != m.log2p || a.in != m.in || a.h != m.h_base || a.nc != m.nc || a.n_in != m.n_in ||
        a.h_n_in != m.h_n_in || a.in_outer != m.in_outer || a.h_outer != m.h_outer || a.n_outer > m.max_outer ||
        !core_tma_supported(a))
        return -1;
    const long long h_need = a.h_mod ? a.h_mod : a.n_outer;
    if (h_need > m.h_outer_count) return -1;
    CoreTmaParams p{};
    p.n_outer = a.n_outer;
    p.h_shift = a.h_shift; p.h_mod = a.h_mod; p.h_off = a.h_off;
    p.scale = a.scale; p.scale_im = a.h_conj ? -a.scale : a.scale; p.gtw = a.gtw; p.gtw_n = a.gtw_n; p.status = status;
    return a.log2p == 8 ? launch_core_tma_t<8>(p, m, a.nc, st) : launch_core_tma_t<10>(p, m, a.nc, st);
}

}  // namespace hn
