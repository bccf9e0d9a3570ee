// Long 1-D path, warp-engine kernels (same decomposition as ct1d.cu: P = P1*P2,
// t = t1*P2 + t2, f = f1 + P1*f2; Appendix B.3 of the paper).
//
//   cols_fwd_w   tile of adjacent column pairs fetched with 16-byte asynchronous copies,
//                one warp-group per column pair: transform along t1 (upper half of the
//                padded input is zero), separate the two real columns, multiply by the
//                inter-pass twiddle, coalesced store of [f1][t2].
//   hspec_w      filter only: transform each kept row along t2 in place and fold in 1/P,
//                so the filter spectrum is computed once per filter, not once per use.
//   core_w       one warp-group per row: transform along t2, multiply by the filter
//                spectrum (Eq. 12), inverse transform chained in registers, undo twiddle.
//   cols_inv_w   rebuild the mirrored half, inverse along f1 keeping t < P/2, crop, gate
//                with q, coalesced store.
#include <type_traits>
#include <cstring>
#include <cstdlib>
#include "common.cuh"
#include "tma_util.cuh"
#include "ct1d.cuh"
#include "plane_util.cuh"

namespace hn {

constexpr int kCtThreads = 256;
// column pairs per tile: at least 16 (64-byte rows of bf16), one or two lines per group of lanes
// line stride of the column kernels: 16-byte aligned and = 2 (mod 16) complex numbers, so that the
// 16-byte accesses of neighbouring lines (tile loads and stores run across lines) hit different banks
__host__ __device__ constexpr int ct_ls(int n) { return (n + 15) / 16 * 16 + 2; }
__host__ __device__ constexpr int ct_tx(int tpl) { return kCtThreads / tpl > 8 ? kCtThreads / tpl : 8; }
// result tile of the forward column kernel as tensor copies: F1 rows in one box, or in two boxes whose
// starts stay on 1024-byte boundaries (rows per box a multiple of 8)
__host__ __device__ constexpr int ct_out_boxes(int f1) { return (f1 + 7) / 8 * 8 > 256 ? 2 : 1; }
__host__ __device__ constexpr int ct_out_box_rows(int f1)
{
    return ct_out_boxes(f1) == 1 ? (f1 + 7) / 8 * 8 : ((f1 + 1) / 2 + 7) / 8 * 8;
}
// the inverse column kernel runs as CTAs of 4 warps: more, smaller tiles in flight per SM
constexpr int kCtInvThreads = 128;
__host__ __device__ constexpr int ct_inv_tx(int tpl) { return kCtInvThreads / tpl > 8 ? kCtInvThreads / tpl : 8; }

template <int BYTES> __device__ __forceinline__ void cp_async_n(void *smem_dst, const void *gmem_src)
{
    const unsigned d = (unsigned)__cvta_generic_to_shared(smem_dst);
    HN_G(gmem_src, BYTES);
    asm volatile("cp.async.ca.shared.global [%0], [%1], %2;\n" ::"r"(d), "l"(gmem_src), "n"(BYTES) : "memory");
}

struct TwoLevelW {
    const float2 *coarse, *fine;
    int lo;
};
__device__ __forceinline__ float2 twp_w(const TwoLevelW &t, unsigned j)
{
    HN_G(t.coarse + (j >> t.lo), 8);
    HN_G(t.fine + (j & ((1u << t.lo) - 1)), 8);
    const float2 c = __ldg(t.coarse + (j >> t.lo));
    const float2 f = __ldg(t.fine + (j & ((1u << t.lo) - 1)));
    return cmul(c, f);
}

// ---- columns, forward ---------------------------------------------------------------------------

struct ColsFwdWArgs {
    const void *a, *b;        // k, v (b == nullptr: plain copy of a, used for a causal filter)
    float2 *out;              // [slices][P1/2+1][P2]
    long long slices;
    long long in_slice;       // elements per slice of the input (multiple of 16 bytes)
    int len;                  // valid elements (<= P/2)
    int *status;              // device word set when a bounded wait on a tensor copy gives up (may be NULL)
    int log2p2;
    const float2 *tw1;        // P1-point table
    TwoLevelW twp;
    bool no_tma;              // development switch: per-thread copies even where tensor copies apply
};

// TMA = true: the tile (all rows t1 of TX column pairs, for k and for v) arrives as tensor copies into
// row-major swizzled buffers, issued by one thread as soon as the previous tile has been read; false: 8-byte
// asynchronous copies per thread into padded rows.
template <typename T, int LOG2P1, bool HAS_B, bool TMA>
__global__ void __launch_bounds__(kCtThreads, (LOG2P1 >= 9 ? 2 : 4))
ct_cols_fwd_w_kernel(ColsFwdWArgs p, const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                     const __grid_constant__ CUtensorMap map_o)
{
    using F = WF<LOG2P1, false>;
    constexpr int P1 = 1 << LOG2P1, HP1 = P1 / 2, F1 = HP1 + 1, TPL = F::TPL;
    constexpr int TX = ct_tx(TPL);                         // column pairs per tile
    constexpr int NGRP = kCtThreads / TPL;                 // groups of lanes per CTA
    constexpr int LS = ct_ls(phys_max(P1) + 2);                // room for the skewed line and for 2*(P1/2+1) bins
    constexpr int PAIRB = 2 * (int)sizeof(T);              // bytes of one column pair of one row
    extern __shared__ float2 smem[];
    float2 *lines = smem;
    float2 *twt = lines + TX * LS;
    // staged inputs [tensor][row t1][pair x], fetched 8 bytes at a time; a row is padded by 8 bytes,
    // which sends the lanes of a group (they differ in t1) to different banks
    constexpr int PG = 8 / PAIRB;                          // column pairs per 8-byte copy
    constexpr int RS = TX * PAIRB + 8;                     // bytes per staged row
    unsigned char *raw = reinterpret_cast<unsigned char *>(twt + P1);
    // tensor copies: rows of TX*PAIRB bytes (64 or 128: the swizzle span), 1024-byte aligned tile buffers
    constexpr unsigned TROW = TX * PAIRB;
    constexpr int TBOXR = HP1 < 256 ? HP1 : 256, TNB = HP1 / TBOXR;
    constexpr unsigned TBYTES = HP1 * TROW;
    static_assert(!TMA || TROW == 64 || TROW == 128, "tile rows match a swizzle span");
    if constexpr (TMA) raw += (1024u - (smem_u32(raw) & 1023u)) & 1023u;
    uint64_t *bar = reinterpret_cast<uint64_t *>(raw + 2 * TBYTES);
    // Result tile as tensor copies too (one line per group): the separated bins are written row-major
    // [f1][pair] into a swizzled staging area that reuses the lines, as two halves of 8 pairs (128-byte rows);
    // boxes of 136 rows keep every box start on a 1024-byte boundary.
    constexpr bool TSTORE = TMA && TX == 16 && NGRP == 16;
    constexpr int ONB = ct_out_boxes(F1), OBOXR = ct_out_box_rows(F1), OHALF = ONB * OBOXR * 128;   // boxes, rows per box, bytes per half
    static_assert(!TSTORE || (F1 <= ONB * OBOXR && 2 * OHALF + 1024 <= TX * LS * 8), "result staging fits the lines");
    unsigned char *to0 = reinterpret_cast<unsigned char *>(lines);
    if constexpr (TSTORE) to0 += (1024u - (smem_u32(to0) & 1023u)) & 1023u;
    const int tid = threadIdx.x, l = tid % TPL, gid = tid / TPL;
    const unsigned m = F::group_mask(tid);
    PassTw<LOG2P1, false>::build(twt, p.tw1, P1, tid, kCtThreads);
    const PassTw<LOG2P1, false> tw{twt};
    const int P2 = 1 << p.log2p2;
    const int tpc = (P2 / 2) / TX;                         // tiles per slice (P2/2 is a multiple of TX)
    const long long tiles = p.slices * tpc;
    const unsigned char *ab = (const unsigned char *)p.a, *bb = (const unsigned char *)p.b;
    auto issue = [&](long long t) {                        // one thread
        const long long s = t / tpc;
        const int x = 2 * (int)(t % tpc) * TX;             // first column of the tile
        mbar_expect_tx(bar, (HAS_B ? 2 : 1) * TBYTES);
#pragma unroll
        for (int b = 0; b < TNB; ++b) {
            tma_load_3d(raw + b * TBOXR * TROW, &map_a, bar, x, b * TBOXR, (int)s);
            if (HAS_B) tma_load_3d(raw + TBYTES + b * TBOXR * TROW, &map_b, bar, x, b * TBOXR, (int)s);
        }
    };
    if constexpr (TMA) {
        if (tid == 0) {
            mbar_init(bar, 1);
            fence_mbar_init();
        }
        __syncthreads();
        if (tid == 0 && (long long)blockIdx.x < tiles) issue(blockIdx.x);
    }
    unsigned phase = 0;
    int failed = 0;
    for (long long t = blockIdx.x; t < tiles; t += gridDim.x, phase ^= 1u) {
        const long long s = t / tpc;
        const int c0 = (int)(t % tpc) * TX;
        const long long base = s * p.in_slice;
        if constexpr (TSTORE) { if (tid == 0) tma_wait_read0(); }   // the previous result tile has left the lines
        __syncthreads();                                   // previous tile done with raw and lines
        if constexpr (TMA) {
            if (!mbar_wait(bar, phase)) failed = 1;
        } else {
        for (int idx = tid; idx < HP1 * (TX / PG); idx += kCtThreads) {
            const int t1 = idx / (TX / PG), xg = idx % (TX / PG);
            const long long e0 = (long long)t1 * P2 + 2 * (c0 + PG * xg);
            unsigned char *d = raw + (size_t)t1 * RS + 8 * xg;
            if (e0 + 2 * PG <= p.len) {
                cp_async_n<8>(d, ab + (base + e0) * sizeof(T));
                if (HAS_B) cp_async_n<8>(d + (size_t)HP1 * RS, bb + (base + e0) * sizeof(T));
            } else {
                for (int e = 0; e < 2 * PG; ++e) {
                    const bool ok = e0 + e < p.len;
                    if (ok) HN_G(reinterpret_cast<const T *>(ab) + base + e0 + e, sizeof(T));
                    if (ok && HAS_B) HN_G(reinterpret_cast<const T *>(bb) + base + e0 + e, sizeof(T));
                    reinterpret_cast<T *>(d)[e] = ok ? reinterpret_cast<const T *>(ab)[base + e0 + e] : T(0.f);
                    if (HAS_B)
                        reinterpret_cast<T *>(d + (size_t)HP1 * RS)[e] = ok ? reinterpret_cast<const T *>(bb)[base + e0 + e] : T(0.f);
                }
            }
        }
        cp_async_wait_all();
        __syncthreads();
        }
        float2 A0[(F1 + TPL - 1) / TPL], A1[(F1 + TPL - 1) / TPL];
        for (int x = gid; x < TX; x += NGRP) {
        float2 *line = lines + x * LS;
        // TMA: the 16-byte chunk of pair x in row idx is XORed with a function of idx that the engine's strides
        // (multiples of 8 rows) leave alone, so it depends on the lane only
        constexpr unsigned RSTR = TMA ? TROW : (unsigned)RS;
        const unsigned sw = TROW == 128 ? ((unsigned)l & 7u) : (((unsigned)l >> 1) & 3u);
        const unsigned xo = TMA ? ((((unsigned)x * PAIRB >> 4) ^ sw) << 4) + (((unsigned)x * PAIRB) & 15u) : (unsigned)x * PAIRB;
        const unsigned char *ra = raw + xo;
        const unsigned char *rb = ra + (TMA ? (size_t)TBYTES : (size_t)HP1 * RS);
        F::template run_to_line<PRUNE_IN>(l, m, tw, line, [&](int, int, int idx) {
            float a0 = staged<T>(ra + (size_t)idx * RSTR, 0, 0), a1 = staged<T>(ra + (size_t)idx * RSTR, 0, 1);
            if (HAS_B) {
                a0 *= staged<T>(rb + (size_t)idx * RSTR, 0, 0);
                a1 *= staged<T>(rb + (size_t)idx * RSTR, 0, 1);
            }
            return make_float2(a0, a1);
        });
        // separate the two real columns, apply W_P^(t2*f1), park both bins in the line
        const unsigned t2 = 2u * (unsigned)(c0 + x);
        {
            // W_P^(t2*f1) with f1 = l + i*TPL is the product of a per-lane factor W_P^(t2*l) (one
            // gathered lookup) and a per-line factor W_P^(t2*TPL*i) (the same address in all lanes)
            // The per-line factor is looked up every fourth step and advanced by W_P^(t2*TPL) in between
            // (at most three products after a table value).
            const float2 cl0 = twp_w(p.twp, t2 * (unsigned)l), cl1 = twp_w(p.twp, (t2 + 1u) * (unsigned)l);
            const float2 st0 = twp_w(p.twp, t2 * (unsigned)TPL), st1 = twp_w(p.twp, (t2 + 1u) * (unsigned)TPL);
            float2 w0 = cl0, w1 = cl1;
#pragma unroll
            for (int i = 0; i < (F1 + TPL - 1) / TPL; ++i) {
                const int f1 = l + i * TPL;
                if (i > 0) {
                    if (i % 4 == 0) {
                        w0 = cmul(cl0, twp_w(p.twp, t2 * (unsigned)(i * TPL)));
                        w1 = cmul(cl1, twp_w(p.twp, (t2 + 1u) * (unsigned)(i * TPL)));
                    } else {
                        w0 = cmul(w0, st0);
                        w1 = cmul(w1, st1);
                    }
                }
                if (f1 < F1) {
                    const float2 z1 = line[F::ph(f1)], z2 = line[F::ph((P1 - f1) & (P1 - 1))];
                    A0[i] = cmul(make_float2(0.5f * (z1.x + z2.x), 0.5f * (z1.y - z2.y)), w0);
                    A1[i] = cmul(make_float2(0.5f * (z1.y + z2.y), 0.5f * (z2.x - z1.x)), w1);
                }
            }
            __syncwarp(m);
            if constexpr (!TSTORE) {
#pragma unroll
                for (int i = 0; i < (F1 + TPL - 1) / TPL; ++i) {
                    const int f1 = l + i * TPL;
                    if (f1 < F1) *reinterpret_cast<float4 *>(line + 2 * f1) = make_float4(A0[i].x, A0[i].y, A1[i].x, A1[i].y);
                }
            }
        }
        }
        if constexpr (TMA) {
            if (__syncthreads_or(failed)) break;           // the tile buffers are free again (and every line has been read)
            if (tid == 0 && t + gridDim.x < tiles) issue(t + gridDim.x);
        } else {
            __syncthreads();
        }
        if constexpr (TSTORE) {
            // group gid holds pair x = gid: rows f1 = l + i*TPL, 16 bytes each, chunk index XORed with (f1 & 7)
            unsigned char *th = to0 + (gid >> 3) * OHALF;
#pragma unroll
            for (int i = 0; i < (F1 + TPL - 1) / TPL; ++i) {
                const int f1 = l + i * TPL;
                if (f1 < F1)
                    *reinterpret_cast<float4 *>(th + f1 * 128 + (((gid & 7) ^ (f1 & 7)) << 4)) = make_float4(A0[i].x, A0[i].y, A1[i].x, A1[i].y);
            }
            fence_async_smem();
            __syncthreads();
            if (tid == 0) {
#pragma unroll
                for (int hh = 0; hh < 2; ++hh)
#pragma unroll
                    for (int rb = 0; rb < ONB; ++rb)
                        tma_store_3d(&map_o, to0 + hh * OHALF + rb * OBOXR * 128, 4 * c0 + 32 * hh, rb * OBOXR, (int)s);
                tma_commit();
            }
            continue;
        }
        float2 *dst = p.out + s * (long long)F1 * P2 + 2 * c0;
        for (int idx = tid; idx < F1 * TX; idx += kCtThreads) {
            const int f1 = idx / TX, x = idx % TX;
            HN_G(dst + (long long)f1 * P2 + 2 * x, 16);
            *reinterpret_cast<float4 *>(dst + (long long)f1 * P2 + 2 * x) =
                *reinterpret_cast<const float4 *>(lines + x * LS + 2 * f1);
        }
    }
    if constexpr (TMA) {
        if (failed) {
            // a wait gave up: say so, then give the copy a bounded time to land before the buffers go away
            if (p.status) atomicExch(p.status, 7);
            mbar_wait(bar, phase);
        }
    }
    if constexpr (TSTORE) { if (tid == 0) tma_wait_all0(); }
}

// ---- filter rows: spectrum in place -----------------------------------------------------------------

struct HspecArgs {
    float2 *h;                // [rows][P2]
    long long rows;
    float scale;
    const float2 *tw2;
};

template <int LOG2P2>
__global__ void __launch_bounds__(256, 2) ct_hspec_w_kernel(HspecArgs p)
{
    using F = WF<LOG2P2, false>;
    constexpr int P2 = 1 << LOG2P2, TPL = F::TPL, G = 256 / TPL, LS = plane_ls(P2);
    extern __shared__ float2 smem[];
    float2 *twt = smem + G * LS;
    const int tid = threadIdx.x, l = tid % TPL, gid = tid / TPL;
    const unsigned m = F::group_mask(tid);
    float2 *line = smem + gid * LS;
    PassTw<LOG2P2, false>::build(twt, p.tw2, P2, tid, 256);
    __syncthreads();
    const PassTw<LOG2P2, false> tw{twt};
    for (long long r = (long long)blockIdx.x * G + gid; r < p.rows; r += (long long)gridDim.x * G) {
        float2 *row = p.h + r * P2;
        F::template run<PRUNE_NONE>(l, m, tw, line,
            [&](int, int, int idx) { HN_G(row + idx, 8); return row[idx]; },
            [&](int, int, int idx, float2 v) { HN_G(row + idx, 8); row[idx] = make_float2(v.x * p.scale, v.y * p.scale); });
        __syncwarp(m);
    }
}

// ---- core --------------------------------------------------------------------------------------------

struct CoreWArgs {
    float2 *u;                // [slices][F1][P2], in place
    const float2 *hspec;      // [filters][F1][P2] spectra along t2 (scaled)
    long long slices;
    int f1n;
    long long h_mod, h_off;
    const float2 *tw2;
    TwoLevelW twp;
};

template <int LOG2P2>
__global__ void __launch_bounds__(256, 2) ct_core_w_kernel(CoreWArgs p)
{
    using F = WF<LOG2P2, false>;
    using FI = WF<LOG2P2, true>;
    constexpr int P2 = 1 << LOG2P2, TPL = F::TPL, NP = F::NP, G = 256 / TPL, LS = plane_ls(P2);
    using PL = typename F::LastPass;
    extern __shared__ float2 smem[];
    float2 *twt = smem + G * LS;
    const int tid = threadIdx.x, l = tid % TPL, gid = tid / TPL;
    const unsigned m = F::group_mask(tid);
    float2 *line = smem + gid * LS;
    PassTw<LOG2P2, false>::build(twt, p.tw2, P2, tid, 256);
    PassTw<LOG2P2, true>::build(twt + P2, p.tw2, P2, tid, 256);
    __syncthreads();
    const PassTw<LOG2P2, false> tw{twt};
    const PassTw<LOG2P2, true> twi{twt + P2};
    const long long rows = p.slices * p.f1n;
    for (long long r = (long long)blockIdx.x * G + gid; r < rows; r += (long long)gridDim.x * G) {
        const long long s = r / p.f1n;
        const int f1 = (int)(r % p.f1n);
        const long long hs = p.h_mod ? (s + p.h_off) % p.h_mod : s;
        float2 *row = p.u + r * P2;
        const float2 *hrow = p.hspec + (hs * p.f1n + f1) * P2;
        // the row is fetched with 16-byte asynchronous copies into the line (two bins per copy)
        for (int c = l; c < P2 / 2; c += TPL) cp_async16(line + 2 * c, row + 2 * c);
        cp_async_wait_all();
        __syncwarp(m);
        float2 Y[PL::IPL][PL::R];
        {
            // first pass reads the unskewed copy, then the usual skewed layout is used
            using P0 = typename F::template Pass<0>;
            float2 keep[P0::IPL][P0::R];
            F::template pass<0, PRUNE_NONE>(l, tw,
                [&](int, int, int idx) { return line[idx]; },
                [&](int i, int rr, int, float2 v) { keep[i][rr] = v; });
            __syncwarp(m);
#pragma unroll
            for (int i = 0; i < P0::IPL; ++i)
#pragma unroll
                for (int rr = 0; rr < P0::R; ++rr) line[F::ph((l + i * TPL) * P0::R + rr)] = keep[i][rr];
            __syncwarp(m);
        }
        F::template mid<1, NP - 1, PRUNE_NONE>(l, m, tw, line);
        F::template pass<NP - 1, PRUNE_NONE>(l, tw,
            [&](int, int, int idx) { return line[F::ph(idx)]; },
            [&](int i, int rr, int, float2 v) { Y[i][rr] = v; });
        // spectral product with the precomputed filter spectrum (coalesced loads, no stores between)
#pragma unroll
        for (int i = 0; i < PL::IPL; ++i)
#pragma unroll
            for (int rr = 0; rr < PL::R; ++rr) {
                HN_G(hrow + F::last_pos(l, i, rr), 8);
                Y[i][rr] = cmul(Y[i][rr], __ldg(hrow + F::last_pos(l, i, rr)));
            }
        __syncwarp(m);
        FI::template pass<0, PRUNE_NONE>(l, twi,
            [&](int i, int rr, int) { return Y[i][rr]; },
            [&](int, int, int idx, float2 v) { line[FI::ph(idx)] = v; });
        __syncwarp(m);
        FI::template mid<1, NP - 1, PRUNE_NONE>(l, m, twi, line);
        // undo the inter-pass twiddle W_P^(t2*f1), t2 = l + TPL*q: per-lane factor W_P^(f1*l) times a
        // per-row factor W_P^(f1*TPL*q) whose address is the same in all lanes
        // (the per-row factor is looked up every fourth leg and advanced by one leg's step in between)
        const float2 cl = twp_w(p.twp, (unsigned)f1 * (unsigned)l);
        using PE = typename FI::LastPass;
        const float2 stp = twp_w(p.twp, (unsigned)f1 * (unsigned)(P2 / PE::R));
        float2 w = cl;
        FI::template pass<NP - 1, PRUNE_NONE>(l, twi,
            [&](int, int, int idx) { return line[FI::ph(idx)]; },
            [&](int, int r, int idx, float2 v) {
                // legs of one item come in order r = 0, 1, ...: positions idx = l + i*TPL + r*(P2/R)
                if (r % 4 == 0) w = cmul(cl, twp_w(p.twp, (unsigned)f1 * (unsigned)(idx - l)));
                else w = cmul(w, stp);
                HN_G(row + idx, 8);
                row[idx] = cmulc(v, w);
            });
        __syncwarp(m);
    }
}

// ---- columns, inverse ------------------------------------------------------------------------------------

struct ColsInvWArgs {
    const float2 *in;         // [slices][F1][P2]
    const void *q;
    void *y;
    long long slices;
    int len;                  // L (multiple of 16 bytes worth of elements)
    int log2p2;
    const float2 *tw1;
    int *status;              // device word set when a bounded wait on a tensor copy gives up (may be NULL)
    bool no_tma;              // development switch: per-thread copies even where tensor copies apply
};

// TMA = true: the gate tile q arrives, and the result tile y leaves, as tensor copies ([t1][pair] rows of
// TX pairs, no swizzle: a warp touches whole consecutive rows); false: per-thread loads and stores.
template <typename T, int LOG2P1, bool TMA>
__global__ void __launch_bounds__(kCtInvThreads, (LOG2P1 >= 9 ? 4 : 8))
ct_cols_inv_w_kernel(ColsInvWArgs p, const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_y)
{
    using FI = WF<LOG2P1, true>;
    constexpr int P1 = 1 << LOG2P1, HP1 = P1 / 2, F1 = HP1 + 1, TPL = FI::TPL;
    constexpr int TX = ct_inv_tx(TPL);
    constexpr int NGRP = kCtInvThreads / TPL;
    constexpr int LS = ct_ls(phys_max(P1) + 2);
    extern __shared__ float2 smem[];
    float2 *lines = smem;
    float2 *twt = lines + TX * LS;
    // gate and result tiles: HP1 rows of TX pairs
    constexpr unsigned QROW = TX * 2 * sizeof(T), QBYTES = HP1 * QROW;
    constexpr int QBOXR = HP1 < 256 ? HP1 : 256, QNB = HP1 / QBOXR;
    unsigned char *tq = reinterpret_cast<unsigned char *>(twt + P1);
    if constexpr (TMA) tq += (128u - (smem_u32(tq) & 127u)) & 127u;
    unsigned char *ty = tq + QBYTES;
    uint64_t *bar = reinterpret_cast<uint64_t *>(ty + QBYTES);
    const int tid = threadIdx.x, l = tid % TPL, gid = tid / TPL;
    const unsigned m = FI::group_mask(tid);
    if constexpr (TMA) {
        if (tid == 0) {
            mbar_init(bar, 1);
            fence_mbar_init();
        }
    }
    unsigned phase = 0;
    int failed = 0;
    PassTw<LOG2P1, true>::build(twt, p.tw1, P1, tid, kCtInvThreads);
    const PassTw<LOG2P1, true> tw{twt};
    const int P2 = 1 << p.log2p2;
    const int tpc = (P2 / 2) / TX;
    const long long tiles = p.slices * tpc;
    const T *pq = (const T *)p.q;
    T *py = (T *)p.y;
    for (long long t = blockIdx.x; t < tiles; t += gridDim.x) {
        const long long s = t / tpc;
        const int c0 = (int)(t % tpc) * TX;
        const float2 *src = p.in + s * (long long)F1 * P2 + 2 * c0;
        if constexpr (TMA) { if (tid == 0) tma_wait_read0(); }        // the previous result tile has left its buffer
        __syncthreads();
        if constexpr (TMA) {
            if (tid == 0) {
                mbar_expect_tx(bar, QBYTES);
#pragma unroll
                for (int b = 0; b < QNB; ++b) tma_load_3d(tq + b * QBOXR * QROW, &map_q, bar, 2 * c0, b * QBOXR, (int)s);
            }
        }
        // both bins of a column pair land side by side in slot f1 of that pair's line
        for (int idx = tid; idx < F1 * TX; idx += kCtInvThreads) {
            const int f1 = idx / TX, x = idx % TX;
            cp_async16(lines + x * LS + 2 * f1, src + (long long)f1 * P2 + 2 * x);
        }
        cp_async_wait_all();
        __syncthreads();
        for (int x = gid; x < TX; x += NGRP) {
            float2 *line = lines + x * LS;
            // legs below half the first-pass radix read bins <= P1/2 directly, the others the mirrored bin
            // conjugated: known per leg at compile time, except where a leg starts at bin P1/2 itself
            constexpr int RH = FI::template Pass<0>::R / 2;
            FI::template run_to_line<PRUNE_OUT, true>(l, m, tw, line, [&](int, int r, int idx) {
                if (r < RH) {
                    const float4 ab = *reinterpret_cast<const float4 *>(line + 2 * idx);
                    return make_float2(ab.x - ab.w, ab.y + ab.z);
                }
                const float4 ab = *reinterpret_cast<const float4 *>(line + 2 * (P1 - idx));
                const float sg = (r == RH && idx == HP1) ? 1.f : -1.f;
                return make_float2(fmaf(-sg, ab.w, ab.x), fmaf(sg, ab.y, ab.z));
            });
        }
        __syncthreads();
        // line x now holds, at position t1 < P1/2, the two real outputs of columns 2x, 2x+1
        const long long base = s * (long long)p.len + 2 * c0;
        // a half warp takes 8 pairs of two neighbouring rows: line stride and skew then spread its
        // 16 reads over all banks, and each row still receives whole 32-byte sectors
        constexpr int NE = HP1 * TX / kCtInvThreads;
        static_assert(HP1 * TX % kCtInvThreads == 0, "whole epilogue rounds");
        const int x = (tid & 7) + 8 * ((tid >> 4) % (TX / 8));
        const int tb = ((tid >> 3) & 1) + 2 * ((tid >> 4) / (TX / 8));
        constexpr int TSTEP = kCtInvThreads / TX;
        using Q2 = typename std::conditional<sizeof(T) == 4, float2, __nv_bfloat162>::type;
        if constexpr (TMA) {
            // gate values from the tile that arrived during the transforms; results into the staging tile
            if (!mbar_wait(bar, phase)) failed = 1;
            phase ^= 1u;
#pragma unroll
            for (int e = 0; e < NE; ++e) {
                const int t1 = tb + e * TSTEP;
                const float2 z = lines[x * LS + FI::ph(t1)];
                const Q2 qv = *reinterpret_cast<const Q2 *>(tq + t1 * QROW + x * sizeof(Q2));
                Q2 *o = reinterpret_cast<Q2 *>(ty + t1 * QROW + x * sizeof(Q2));
                if constexpr (sizeof(T) == 4) *o = make_float2(z.x * qv.x, z.y * qv.y);
                else *o = __floats2bfloat162_rn(z.x * __low2float(qv), z.y * __high2float(qv));
            }
            fence_async_smem();
            if (__syncthreads_or(failed)) break;
            if (tid == 0) {
#pragma unroll
                for (int b = 0; b < QNB; ++b) tma_store_3d(&map_y, ty + b * QBOXR * QROW, 2 * c0, b * QBOXR, (int)s);
                tma_commit();
            }
            continue;
        }
        // gate values first (all requests in flight together), then products and stores
        const long long ox = base + 2 * x;
        Q2 qv[NE];
#pragma unroll
        for (int e = 0; e < NE; ++e) {
            const int t1 = tb + e * TSTEP;
            const long long tt = (long long)t1 * P2 + 2 * (c0 + x);
            if (tt < p.len) HN_G(pq + ox + (long long)t1 * P2, 2 * sizeof(T));
            if (tt < p.len) qv[e] = __ldg(reinterpret_cast<const Q2 *>(pq + ox + (long long)t1 * P2));
        }
#pragma unroll
        for (int e = 0; e < NE; ++e) {
            const int t1 = tb + e * TSTEP;
            const long long tt = (long long)t1 * P2 + 2 * (c0 + x);
            if (tt < p.len) {
                const float2 z = lines[x * LS + FI::ph(t1)];
                const long long o = ox + (long long)t1 * P2;
                HN_G(py + o, 2 * sizeof(T));
                if constexpr (sizeof(T) == 4) {
                    *reinterpret_cast<float2 *>(py + o) = make_float2(z.x * qv[e].x, z.y * qv[e].y);
                } else {
                    *reinterpret_cast<__nv_bfloat162 *>(py + o) =
                        __floats2bfloat162_rn(z.x * __low2float(qv[e]), z.y * __high2float(qv[e]));
                }
            }
        }
    }
    if constexpr (TMA) {
        if (failed) {
            if (p.status) atomicExch(p.status, 8);
            mbar_wait(bar, phase ^ 1u);
        }
        if (tid == 0) tma_wait_all0();
    }
}

// ---- launchers ----------------------------------------------------------------------------------------------

static int ctw_sms()
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

bool ct1d_w_supported(int log2p1, int log2p2, int L, int K, int causal, int dtype)
{
    const int es = dtype == 0 ? 4 : 2;
    if (log2p1 < 7 || log2p1 > 10 || log2p2 < 7 || log2p2 > 10) return false;
    if (((long long)L * es) % 16 != 0) return false;               // 16-byte copies of whole chunks
    if (causal && ((long long)K * es) % 16 != 0) return false;
    const int tx = ct_tx(log2p1 >= 10 ? 32 : (log2p1 >= 8 ? 16 : 8));
    if (((1 << log2p2) / 2) % tx != 0) return false;
    return true;
}

template <typename T, int LOG2P1, bool HAS_B, bool TMA>
static void launch_cols_fwd_w_tt(const ColsFwdWArgs &a, const CUtensorMap &ma, const CUtensorMap &mb, const CUtensorMap &mo, int grid,
                                size_t sm, cudaStream_t st)
{
    static DevOnce attr;
    if (attr.first())
        cudaFuncSetAttribute(ct_cols_fwd_w_kernel<T, LOG2P1, HAS_B, TMA>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
    ct_cols_fwd_w_kernel<T, LOG2P1, HAS_B, TMA><<<grid, kCtThreads, sm, st>>>(a, ma, mb, mo);
}

template <typename T, int LOG2P1> static int launch_cols_fwd_w_t(const ColsFwdWArgs &a, cudaStream_t st)
{
    using F = WF<LOG2P1, false>;
    constexpr int P1 = 1 << LOG2P1, TX = ct_tx(F::TPL), LS = ct_ls(phys_max(P1) + 2);
    const size_t sm = sizeof(float2) * ((size_t)TX * LS + P1) + (size_t)2 * (P1 / 2) * (2 * TX * sizeof(T) + 8);
    const int P2 = 1 << a.log2p2;
    const long long tiles = a.slices * ((P2 / 2) / TX);
    const long long res = (LOG2P1 >= 9 ? 2ll : 4ll) * ctw_sms();   // resident CTAs
    const int grid = (int)(tiles < res ? tiles : res);
    if (grid <= 0) return 0;
    // Tensor copies need the slice to be a whole number of rows of P2 elements (then [slice][row][P2] is an
    // exact view of the input and rows past the data read as zeros) and tile rows of 64 or 128 bytes.
    alignas(64) CUtensorMap ma, mb, mo;
    memset(&ma, 0, sizeof(ma));
    memset(&mb, 0, sizeof(mb));
    memset(&mo, 0, sizeof(mo));
    constexpr unsigned TROW = TX * 2 * sizeof(T);
    bool tma = (TROW == 64 || TROW == 128) && a.len % P2 == 0 && a.slices < (1ll << 31) && tma_available() && !a.no_tma;
    if (tma) {
        constexpr int HP1 = P1 / 2;
        const unsigned long long dims[3] = {(unsigned long long)P2, (unsigned long long)(a.len / P2), (unsigned long long)a.slices};
        const unsigned long long strides[2] = {(unsigned long long)P2 * sizeof(T), (unsigned long long)a.in_slice * sizeof(T)};
        const unsigned box[3] = {2 * TX, (unsigned)(HP1 < 256 ? HP1 : 256), 1};
        tma = tma_encode_3d_cached(&ma, a.a, sizeof(T) == 2, dims, strides, box, (int)TROW);
        if (tma && a.b) tma = tma_encode_3d_cached(&mb, a.b, sizeof(T) == 2, dims, strides, box, (int)TROW);
        // results [slice][P1/2+1][P2] complex, as fp32: boxes of 8 column pairs (32 floats) by 136 rows
        const unsigned long long od[3] = {2ull * P2, (unsigned long long)(HP1 + 1), (unsigned long long)a.slices};
        const unsigned long long os[2] = {(unsigned long long)P2 * 8, (unsigned long long)(HP1 + 1) * P2 * 8};
        const unsigned ob[3] = {32, (unsigned)ct_out_box_rows(HP1 + 1), 1};
        if (tma) tma = tma_encode_3d_cached(&mo, a.out, false, od, os, ob, 128);
    }
    if constexpr (TROW == 64 || TROW == 128) {
        if (tma) {
            if (a.b) launch_cols_fwd_w_tt<T, LOG2P1, true, true>(a, ma, mb, mo, grid, sm, st);
            else launch_cols_fwd_w_tt<T, LOG2P1, false, true>(a, ma, mb, mo, grid, sm, st);
            return 1;
        }
    }
    if (a.b) launch_cols_fwd_w_tt<T, LOG2P1, true, false>(a, ma, mb, mo, grid, sm, st);
    else launch_cols_fwd_w_tt<T, LOG2P1, false, false>(a, ma, mb, mo, grid, sm, st);
    return 1;
}

template <typename T, int LOG2P1, bool TMA>
static void launch_cols_inv_w_tt(const ColsInvWArgs &a, const CUtensorMap &mq, const CUtensorMap &my, int grid, size_t sm, cudaStream_t st)
{
    static DevOnce attr;
    if (attr.first())
        cudaFuncSetAttribute(ct_cols_inv_w_kernel<T, LOG2P1, TMA>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
    ct_cols_inv_w_kernel<T, LOG2P1, TMA><<<grid, kCtInvThreads, sm, st>>>(a, mq, my);
}

template <typename T, int LOG2P1> static int launch_cols_inv_w_t(const ColsInvWArgs &a, cudaStream_t st)
{
    using F = WF<LOG2P1, true>;
    constexpr int P1 = 1 << LOG2P1, HP1 = P1 / 2, TX = ct_inv_tx(F::TPL), LS = ct_ls(phys_max(P1) + 2);
    constexpr unsigned QROW = TX * 2 * sizeof(T);
    // lines, twiddles, and (tensor-copy variant) gate tile, result tile, barrier, alignment slack
    const size_t sm = sizeof(float2) * ((size_t)TX * LS + P1) + 2 * (size_t)HP1 * QROW + 8 + 128;
    const int P2 = 1 << a.log2p2;
    const long long tiles = a.slices * ((P2 / 2) / TX);
    const long long res = (LOG2P1 >= 9 ? 4ll : 8ll) * ctw_sms();   // resident CTAs
    const int grid = (int)(tiles < res ? tiles : res);
    if (grid <= 0) return 0;
    alignas(64) CUtensorMap mq, my;
    memset(&mq, 0, sizeof(mq));
    memset(&my, 0, sizeof(my));
    // tensor copies need the slice to be a whole number of rows of P2 elements
    bool tma = a.len % P2 == 0 && a.slices < (1ll << 31) && QROW % 16 == 0 && tma_available() && !a.no_tma;
    if (tma) {
        const unsigned long long dims[3] = {(unsigned long long)P2, (unsigned long long)(a.len / P2), (unsigned long long)a.slices};
        const unsigned long long strides[2] = {(unsigned long long)P2 * sizeof(T), (unsigned long long)a.len * sizeof(T)};
        const unsigned box[3] = {2 * TX, (unsigned)(HP1 < 256 ? HP1 : 256), 1};
        tma = tma_encode_3d_cached(&mq, a.q, sizeof(T) == 2, dims, strides, box, 0) && tma_encode_3d_cached(&my, a.y, sizeof(T) == 2, dims, strides, box, 0);
    }
    if (tma) launch_cols_inv_w_tt<T, LOG2P1, true>(a, mq, my, grid, sm, st);
    else launch_cols_inv_w_tt<T, LOG2P1, false>(a, mq, my, grid, sm, st);
    return 1;
}

template <int LOG2P2> static int launch_rows_w_t(const HspecArgs *hs, const CoreWArgs *co, cudaStream_t st)
{
    using F = WF<LOG2P2, false>;
    constexpr int P2 = 1 << LOG2P2, G = 256 / F::TPL, LS = plane_ls(P2);
    const size_t sm = sizeof(float2) * ((size_t)G * LS + 2 * P2);
    static DevOnce attr;
    if (attr.first()) {
        cudaFuncSetAttribute(ct_hspec_w_kernel<LOG2P2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
        cudaFuncSetAttribute(ct_core_w_kernel<LOG2P2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
    }
    const long long rows = hs ? hs->rows : co->slices * co->f1n;
    const long long want = (rows + G - 1) / G;
    const int grid = (int)(want < (long long)ctw_sms() * 2 ? want : (long long)ctw_sms() * 2);
    if (grid <= 0) return 0;
    if (hs) ct_hspec_w_kernel<LOG2P2><<<grid, 256, sm, st>>>(*hs);
    else ct_core_w_kernel<LOG2P2><<<grid, 256, sm, st>>>(*co);
    return 1;
}

#define HN_SWITCH_CTW(x, CALL)                                                                  \
    switch (x) {                                                                                \
    case 7: CALL(7); break; case 8: CALL(8); break; case 9: CALL(9); break; case 10: CALL(10); break; \
    default: return -1;                                                                         \
    }

static int launch_rows_w(int log2p2, const HspecArgs *hs, const CoreWArgs *co, cudaStream_t st)
{
    int n = 0;
#define CALLR(L) n = launch_rows_w_t<L>(hs, co, st)
    HN_SWITCH_CTW(log2p2, CALLR)
#undef CALLR
    return n;
}

int ct1d_w_filter(Ct1dPlan *c, const void *h, long long n, bool staged_ok, cudaStream_t st, int *launches, Prof *prof,
                  int (*fallback)(Ct1dPlan *, const char *, long long, cudaStream_t, int *, Prof *))
{
    const TwoLevelW twp{c->twp_coarse, c->twp_fine, c->lo};
    if (staged_ok) {
        ColsFwdWArgs a{};
        a.a = h; a.b = nullptr; a.out = c->wh; a.slices = n; a.in_slice = c->K; a.len = c->K; a.status = c->status; a.no_tma = c->sw.no_tma;
        a.log2p2 = c->log2p2; a.tw1 = c->tw1; a.twp = twp;
        prof->begin(KID_CT_COLS_H, st);
        int r = 0;
#define CALLF(L) r = launch_cols_fwd_w_t<float, L>(a, st)
#define CALLB(L) r = launch_cols_fwd_w_t<bf16, L>(a, st)
        if (c->dt_h == 0) { HN_SWITCH_CTW(c->log2p1, CALLF) } else { HN_SWITCH_CTW(c->log2p1, CALLB) }
#undef CALLF
#undef CALLB
        prof->end(st);
        if (r < 0) return -1;
        *launches += r;
    } else if (fallback(c, (const char *)h, n, st, launches, prof)) {
        return -1;
    }
    HspecArgs hs{};
    hs.h = c->wh; hs.rows = n * ((1 << c->log2p1) / 2 + 1); hs.scale = (float)ldexp(1.0, -c->log2p); hs.tw2 = c->tw2;
    prof->begin(KID_CT_HSPEC, st);
    int r = launch_rows_w(c->log2p2, &hs, nullptr, st);
    prof->end(st);
    if (r < 0) return -1;
    *launches += r;
    return 0;
}

int ct1d_w_body(Ct1dPlan *c, const void *q, const void *k, const void *v, long long n, bool shared, long long s0,
                void *y, cudaStream_t st, int *launches, Prof *prof)
{
    const TwoLevelW twp{c->twp_coarse, c->twp_fine, c->lo};
    ColsFwdWArgs a{};
    a.a = k; a.b = v; a.out = c->wu; a.slices = n; a.in_slice = c->L; a.len = c->L; a.status = c->status; a.no_tma = c->sw.no_tma;
    a.log2p2 = c->log2p2; a.tw1 = c->tw1; a.twp = twp;
    prof->begin(KID_CT_COLS_U, st);
    int r = 0;
#define CALLF(L) r = launch_cols_fwd_w_t<float, L>(a, st)
#define CALLB(L) r = launch_cols_fwd_w_t<bf16, L>(a, st)
    if (c->dt_in == 0) { HN_SWITCH_CTW(c->log2p1, CALLF) } else { HN_SWITCH_CTW(c->log2p1, CALLB) }
#undef CALLF
#undef CALLB
    prof->end(st);
    if (r < 0) return -1;
    *launches += r;
    CoreWArgs co{};
    co.u = c->wu; co.hspec = c->wh; co.slices = n; co.f1n = (1 << c->log2p1) / 2 + 1;
    co.h_mod = shared ? c->C : 0; co.h_off = shared ? s0 % c->C : 0;
    co.tw2 = c->tw2; co.twp = twp;
    prof->begin(KID_CT_CORE, st);
    r = launch_rows_w(c->log2p2, nullptr, &co, st);
    prof->end(st);
    if (r < 0) return -1;
    *launches += r;
    ColsInvWArgs ci{};
    ci.in = c->wu; ci.q = q; ci.y = y; ci.slices = n; ci.len = c->L; ci.log2p2 = c->log2p2; ci.tw1 = c->tw1; ci.status = c->status; ci.no_tma = c->sw.no_tma;
    prof->begin(KID_CT_COLS_INV, st);
#define CALLF(L) r = launch_cols_inv_w_t<float, L>(ci, st)
#define CALLB(L) r = launch_cols_inv_w_t<bf16, L>(ci, st)
    if (c->dt_out == 0) { HN_SWITCH_CTW(c->log2p1, CALLF) } else { HN_SWITCH_CTW(c->log2p1, CALLB) }
#undef CALLF
#undef CALLB
    prof->end(st);
    if (r < 0) return -1;
    *launches += r;
    return 0;
}

}  // namespace hn
