// Fused spectral core along a strided axis for 256-point lines, tiles moved by TMA.
//
// Same arithmetic as core_w.cu (forward transform of the filter lines, forward transform of the
// k*v lines, spectral product of Eq. 12 of the paper, inverse, cropped half written back in
// place), but the tiles -- 16 adjacent bins by all rows of the axis -- travel as tensor copies:
//
//   cp.async.bulk.tensor loads   filter tile (two boxes of 128 rows: the wrapped placement of the
//                                taps is two row ranges) and k*v tile (one box; rows past the data
//                                and bins past the end come back as zeros)
//   cp.async.bulk.tensor store   the cropped result tile
//
// One elected thread issues them; nobody computes addresses or waits per element.  The boxes land
// row-major (128 bytes per row) with the 128-byte swizzle, which spreads the 16 rows a group of
// lanes reads at once over 8 bank groups.  A tile buffer is free again as soon as the first pass
// has read it, so the next tile's copy runs under the rest of this tile's arithmetic.
//
// Every wait on a copy is bounded: if a barrier does not complete, the CTA records it in the
// status word, waits (bounded again) for what is still in flight and returns.
#include <cuda.h>
#include <cstdint>
#include "common.cuh"
#include "plane_util.cuh"
#include "core_tma.cuh"

namespace hn {

constexpr int kTmaLog2 = 8;
constexpr int kTmaN = 1 << kTmaLog2;                 // line length
constexpr int kTmaThreads = 256;
constexpr int kTmaTX = 16;                           // bins per tile (one 128-byte row)
constexpr int kTmaHalf = kTmaN / 2;                  // rows per box
constexpr unsigned kRowBytes = kTmaTX * 8;           // 128
constexpr unsigned kBoxBytes = kTmaHalf * kRowBytes; // 16 KB
constexpr int kWaitLimit = 1 << 22;                  // polls of a barrier before giving up

__device__ __forceinline__ unsigned smem_u32(const void *p) { return (unsigned)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t *b, unsigned count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(smem_u32(b)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *b, unsigned bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(smem_u32(b)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *b, unsigned parity)
{
    unsigned ok;
    asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
                 : "=r"(ok) : "r"(smem_u32(b)), "r"(parity) : "memory");
    return ok != 0;
}
// bounded wait; false if the phase did not complete
__device__ __forceinline__ bool mbar_wait(uint64_t *b, unsigned parity)
{
    for (int i = 0; i < kWaitLimit; ++i)
        if (mbar_try_wait(b, parity)) return true;
    return false;
}
__device__ __forceinline__ void tma_load_3d(void *dst, const CUtensorMap *map, uint64_t *bar, int x, int y, int z)
{
    asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];\n"
                 ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(x), "r"(y), "r"(z) : "memory");
}
__device__ __forceinline__ void tma_store_3d(const CUtensorMap *map, const void *src, int x, int y, int z)
{
    asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];\n"
                 ::"l"(map), "r"(smem_u32(src)), "r"(x), "r"(y), "r"(z) : "memory");
}
__device__ __forceinline__ void tma_commit() { asm volatile("cp.async.bulk.commit_group;\n" ::: "memory"); }
__device__ __forceinline__ void tma_wait_read0() { asm volatile("cp.async.bulk.wait_group.read 0;\n" ::: "memory"); }
__device__ __forceinline__ void tma_wait_all0() { asm volatile("cp.async.bulk.wait_group 0;\n" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory"); }
__device__ __forceinline__ void fence_mbar_init() { asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory"); }

struct CoreTmaParams {
    long long n_outer;
    int tiles_per_outer;      // ceil(nc / 16)
    int h_shift;              // filter row (pos + h_shift) mod N sits at position pos
    long long h_mod, h_off;   // filter outer index = h_mod ? (o + h_off) % h_mod : o
    float scale;
    const float2 *gtw;
    int gtw_n;
    int *status;              // device word: 0 ok, else which wait gave up
};

// shared memory: tile buffers first (1024-byte aligned, as the swizzle pattern repeats every 8 rows)
struct CoreTmaSmem {
    static constexpr int LS = line_stride(kTmaN);
    static constexpr size_t TH = 0;                                  // filter tile, 256 rows
    static constexpr size_t TU = TH + 2 * kBoxBytes;                 // k*v tile, 128 rows
    static constexpr size_t TO = TU + kBoxBytes;                     // result tile, 128 rows
    static constexpr size_t LINES = TO + kBoxBytes;                  // one skewed line per group
    static constexpr size_t TW = LINES + sizeof(float2) * kTmaTX * LS;
    static constexpr size_t BARS = TW + sizeof(float2) * kTmaN;
    static constexpr size_t TOTAL = BARS + 2 * sizeof(uint64_t) + 1024;    // + room to align the start
};

__global__ void __launch_bounds__(kTmaThreads, 2)
axis_core_tma_kernel(const __grid_constant__ CUtensorMap map_u, const __grid_constant__ CUtensorMap map_h, CoreTmaParams p)
{
    using F = WF<kTmaLog2, false>;
    using FI = WF<kTmaLog2, true>;
    constexpr int N = kTmaN, TPL = F::TPL, NP = F::NP;
    static_assert(TPL == 16 && NP == 2 && kTmaThreads / TPL == kTmaTX, "tile = one line per group of 16 lanes");
    using PL = typename F::template Pass<NP - 1>;
    using PE = typename FI::template Pass<NP - 1>;
    extern __shared__ __align__(1024) unsigned char smem_dyn[];
    // the swizzle pattern is a function of the shared-memory address: start on a 1024-byte boundary
    unsigned char *smem_raw = smem_dyn + ((1024u - (smem_u32(smem_dyn) & 1023u)) & 1023u);
    unsigned char *th = smem_raw + CoreTmaSmem::TH;
    unsigned char *tu = smem_raw + CoreTmaSmem::TU;
    unsigned char *to = smem_raw + CoreTmaSmem::TO;
    float2 *lines = reinterpret_cast<float2 *>(smem_raw + CoreTmaSmem::LINES);
    float2 *twt = reinterpret_cast<float2 *>(smem_raw + CoreTmaSmem::TW);
    uint64_t *bar_h = reinterpret_cast<uint64_t *>(smem_raw + CoreTmaSmem::BARS);
    uint64_t *bar_u = bar_h + 1;
    const int tid = threadIdx.x, l = tid % TPL, gid = tid / TPL;
    const unsigned m = F::group_mask(tid);
    float2 *line = lines + gid * CoreTmaSmem::LS;
    for (int t = tid; t < N; t += kTmaThreads) twt[t] = p.gtw[t * (p.gtw_n / N)];
    if (tid == 0) {
        mbar_init(bar_h, 1);
        mbar_init(bar_u, 1);
        fence_mbar_init();
    }
    __syncthreads();
    PlaneTw<kTmaLog2, false> tw;
    tw.init(l, twt, twt, tid, kTmaThreads);            // 16 x 16: twiddles live in registers, no table
    static_assert(PlaneTw<kTmaLog2, false>::HOIST && PlaneTw<kTmaLog2, true>::HOIST, "register twiddles");
    PlaneTw<kTmaLog2, true> twi;
    twi.init(l, twt, twt, tid, kTmaThreads);
    // Row z = l + 16 r of bin `gid` inside a swizzled tile: 128 bytes per row, the 16-byte chunk index
    // is XORed with (z & 7) = (l & 7), so every r is the same per-lane offset plus r * 2048 bytes.
    const unsigned tile_off = (unsigned)l * kRowBytes + ((((unsigned)gid >> 1) ^ ((unsigned)l & 7u)) << 4) + ((unsigned)gid & 1u) * 8u;
    const long long tiles = p.n_outer * p.tiles_per_outer;
    auto issue_h = [&](long long t) {                  // one thread
        const long long o = t / p.tiles_per_outer;
        const int x = (int)(t % p.tiles_per_outer) * kTmaTX * 2;          // in floats
        const long long oh = p.h_mod ? (o + p.h_off) % p.h_mod : o;
        mbar_expect_tx(bar_h, 2 * kBoxBytes);
        tma_load_3d(th, &map_h, bar_h, x, p.h_shift, (int)oh);                        // positions [0, 128)
        tma_load_3d(th + kBoxBytes, &map_h, bar_h, x, p.h_shift - kTmaHalf, (int)oh); // positions [128, 256)
    };
    auto issue_u = [&](long long t) {
        const long long o = t / p.tiles_per_outer;
        const int x = (int)(t % p.tiles_per_outer) * kTmaTX * 2;
        mbar_expect_tx(bar_u, kBoxBytes);
        tma_load_3d(tu, &map_u, bar_u, x, 0, (int)o);
    };
    long long t = blockIdx.x;
    if (tid == 0 && t < tiles) { issue_h(t); issue_u(t); }
    unsigned phase = 0;
    int failed = 0;
    for (; t < tiles; t += gridDim.x, phase ^= 1u) {
        const long long tn = t + gridDim.x;
        float2 H[PL::IPL][PL::R];
        // ---- filter lines: tile -> registers ------------------------------------------------------
        if (!mbar_wait(bar_h, phase)) failed = 1;
        {
            const float2 *src = reinterpret_cast<const float2 *>(th + tile_off);
            F::template pass<0, PRUNE_NONE>(l, tw,
                [&](int, int r, int) { return src[r * (2048 / 8)]; },
                [&](int, int, int idx, float2 v) { line[F::ph(idx)] = v; });
        }
        if (__syncthreads_or(failed)) break;           // the filter tile buffer is free again
        if (tid == 0 && tn < tiles) issue_h(tn);
        F::template pass<NP - 1, PRUNE_NONE>(l, tw,
            [&](int, int, int idx) { return line[F::ph(idx)]; },
            [&](int i, int r, int, float2 v) { H[i][r] = make_float2(v.x * p.scale, v.y * p.scale); });
        __syncwarp(m);
        // ---- k*v lines: tile -> spectrum, product, inverse ----------------------------------------
        if (!mbar_wait(bar_u, phase)) failed = 2;
        {
            const float2 *src = reinterpret_cast<const float2 *>(tu + tile_off);
            F::template pass<0, PRUNE_IN>(l, tw,
                [&](int, int r, int) { return src[r * (2048 / 8)]; },
                [&](int, int, int idx, float2 v) { line[F::ph(idx)] = v; });
        }
        if (tid == 0) tma_wait_read0();                // the previous result tile has left its buffer
        if (__syncthreads_or(failed)) break;           // the k*v tile buffer is free again
        if (tid == 0 && tn < tiles) issue_u(tn);
        float2 Y[PL::IPL][PL::R];
        F::template pass<NP - 1, PRUNE_NONE>(l, tw,
            [&](int, int, int idx) { return line[F::ph(idx)]; },
            [&](int i, int r, int, float2 v) { Y[i][r] = cmul(v, H[i][r]); });
        __syncwarp(m);
        FI::template pass<0, PRUNE_NONE>(l, twi,
            [&](int i, int r, int) { return Y[i][r]; },
            [&](int, int, int idx, float2 v) { line[FI::ph(idx)] = v; });
        __syncwarp(m);
        {
            float2 *dst = reinterpret_cast<float2 *>(to + tile_off);
            FI::template pass<NP - 1, PRUNE_OUT>(l, twi,
                [&](int, int, int idx) { return line[FI::ph(idx)]; },
                [&](int, int r, int, float2 v) { dst[r * (2048 / 8)] = v; });
        }
        __syncwarp(m);
        fence_async_smem();                            // generic-proxy writes visible to the copy engine
        __syncthreads();
        if (tid == 0) {
            const long long o = t / p.tiles_per_outer;
            const int x = (int)(t % p.tiles_per_outer) * kTmaTX * 2;
            tma_store_3d(&map_u, to, x, 0, (int)o);
            tma_commit();
        }
    }
    if (failed || t < tiles) {
        // a wait gave up: say so, then give copies that may still be in flight a bounded time to land
        if (failed) atomicExch(p.status, failed);
        mbar_wait(bar_h, phase);
        mbar_wait(bar_u, phase);
    }
    if (tid == 0) tma_wait_all0();
}

// ---- host side -------------------------------------------------------------------------------------------

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult qr;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qr) == cudaSuccess &&
            qr == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
        else
            cudaGetLastError();
    }
    return fn;
}

// [outer][rows][nc] complex fp32, seen as fp32 with 2*nc entries per row; box = 32 floats x 128 rows
static bool make_map(CUtensorMap *map, const float2 *base, long long outer, int rows, int nc, long long outer_stride_elems)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[3] = {(cuuint64_t)2 * nc, (cuuint64_t)rows, (cuuint64_t)outer};
    const cuuint64_t strides[2] = {(cuuint64_t)nc * 8, (cuuint64_t)outer_stride_elems * 8};
    const cuuint32_t box[3] = {(cuuint32_t)kTmaTX * 2, (cuuint32_t)kTmaHalf, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    if ((strides[0] % 16) || (strides[1] % 16) || ((uintptr_t)base % 16)) return false;
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<float2 *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool core_tma_supported(const AxisArgs &a)
{
    return a.log2p == kTmaLog2 && a.in == a.out && a.in_outer == a.out_outer && a.n_in == a.n_out &&
           a.n_in >= 1 && a.n_in <= kTmaHalf && a.h_n_in >= 1 && a.h_n_in <= kTmaN && a.shift == 0 &&
           a.h_shift >= 0 && a.h_shift < kTmaN && (a.nc % 2) == 0 && a.n_outer < (1ll << 31) && encode_fn() != nullptr;
}

bool core_tma_make(CoreTmaMaps *m, const AxisArgs &a, long long max_outer, long long h_outer_count)
{
    m->valid = false;
    if (!core_tma_supported(a)) return false;
    static_assert(sizeof(m->u) >= sizeof(CUtensorMap) && sizeof(m->h) >= sizeof(CUtensorMap), "room for a tensor map");
    if (!make_map(reinterpret_cast<CUtensorMap *>(m->u), a.in, max_outer, a.n_in, a.nc, a.in_outer)) return false;
    if (!make_map(reinterpret_cast<CUtensorMap *>(m->h), a.h, h_outer_count, a.h_n_in, a.nc, a.h_outer)) return false;
    m->in = a.in; m->h_base = a.h; m->nc = a.nc; m->n_in = a.n_in; m->h_n_in = a.h_n_in;
    m->in_outer = a.in_outer; m->h_outer = a.h_outer; m->max_outer = max_outer; m->h_outer_count = h_outer_count;
    m->valid = true;
    return true;
}

int launch_core_tma(const AxisArgs &a, const CoreTmaMaps &m, int *status, cudaStream_t st)
{
    // the maps describe fixed buffers: refuse anything else
    if (!m.valid || a.in != m.in || a.h != m.h_base || a.nc != m.nc || a.n_in != m.n_in || a.h_n_in != m.h_n_in ||
        a.in_outer != m.in_outer || a.h_outer != m.h_outer || a.n_outer > m.max_outer || !core_tma_supported(a))
        return -1;
    const long long h_need = a.h_mod ? a.h_mod : a.n_outer;
    if (h_need > m.h_outer_count) return -1;
    CoreTmaParams p{};
    p.n_outer = a.n_outer;
    p.tiles_per_outer = (a.nc + kTmaTX - 1) / kTmaTX;
    p.h_shift = a.h_shift; p.h_mod = a.h_mod; p.h_off = a.h_off;
    p.scale = a.scale; p.gtw = a.gtw; p.gtw_n = a.gtw_n; p.status = status;
    static int sms = 0;
    if (!sms) {
        int dev = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (sms <= 0) sms = 148;
    }
    static DevOnce attr;
    if (attr.first())
        cudaFuncSetAttribute(axis_core_tma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)CoreTmaSmem::TOTAL);
    const long long tiles = p.n_outer * p.tiles_per_outer;
    const int grid = (int)(tiles < 2ll * sms ? tiles : 2ll * sms);
    if (grid <= 0) return 0;
    axis_core_tma_kernel<<<grid, kTmaThreads, CoreTmaSmem::TOTAL, st>>>(
        *reinterpret_cast<const CUtensorMap *>(m.u), *reinterpret_cast<const CUtensorMap *>(m.h), p);
    return 1;
}

}  // namespace hn
