// Kernel synthesis: the input-dependent convolution kernel K(x) of HyenaND evaluated on the tap grid,
//
//     K(x)[b, c, i] = w_c(c_i) * f_theta(c_i; gamma_b, beta_b)[c]
//
// f_theta a SIREN with a learnable frequency vector (Eq. 3 of the paper), FiLM-modulated per batch entry (Eq. 4),
// w the per-channel, per-axis Gaussian window (Eq. 6) or, for causal 1-D kernels, the exponential window of
// Appendix A.3.  One thread evaluates the network at NC neighbouring taps: the hidden activations stay in
// registers, the weights are read from shared memory as 16-byte broadcasts (every lane reads the same address), so
// each loaded weight feeds NC fused multiply-adds.  The output layer runs over chunks of channels whose weights are
// staged in shared memory in turn; for a fixed channel a warp stores 32*NC neighbouring taps (coalesced).
// Sines: the first layer's arguments reach tens of radians, where the hardware sine alone loses accuracy, so every
// argument is first reduced to [-pi, pi] with a two-term 2*pi (exact to fp32 rounding for the multiples that occur);
// the hardware sine's absolute error on that interval is 2^-21.4.  This translation unit is compiled without
// fast-math so that nothing else (divisions, the reduction) is replaced by approximations.
#include "common.cuh"
#include "synth.cuh"
#include "tma_util.cuh"
#include "tmem_util.cuh"
#include <type_traits>

namespace hn {

// parameter loads (checked in the checked build)
#define SYN_LD(ptr, idx) (HN_G((ptr) + (idx), 4), (ptr)[idx])

constexpr int kSynThreads = 128;
constexpr int kSynChanChunk = 32;        // output channels whose weights sit in shared memory at a time

__device__ __forceinline__ float sin_reduced(float x)
{
    // nearest integer of x / 2 pi by adding and subtracting 1.5 * 2^23 (two full-rate additions; the rounding
    // instruction runs on the quarter-rate pipe the sine itself needs); exact for |x / 2 pi| < 2^22
    const float k = (fmaf(x, 0.15915494309189535f, 12582912.f)) - 12582912.f;
    float r = fmaf(-k, 6.2831854820251465f, x);           // float(2 pi)
    r = fmaf(k, 1.7484555e-7f, r);                        // float(2 pi) - 2 pi
    return __sinf(r);
}

__device__ __forceinline__ float axis_coord(int m, int L, int mode)
{
    if (L <= 1) return 0.f;
    if (mode == 0) return (float)(m - (L - 1)) / (float)(L - 1);
    if (mode == 1) return (float)m / (float)(L - 1);
    const int d = 2 * m <= L ? m : m - L;
    return (float)d / (0.5f * (float)L);
}

template <typename T, int HF, int NC>
__global__ void __launch_bounds__(kSynThreads) synth_kernel(SynthArgs p)
{
    extern __shared__ float4 smem4[];
    float *sm = reinterpret_cast<float *>(smem4);
    const int J = p.layers, H = p.hidden, N = p.ndim;
    // shared memory: W1 [HF][4] (x, y, z coefficient, bias), omega [HF], hidden layers [J-1][HF][HF] + bias [J-1][HF],
    // FiLM [J][2][HF], output chunk [kSynChanChunk][HF] + bias + window parameters
    float *sW1 = sm;
    float *sOm = sW1 + HF * 4;
    float *sWh = sOm + HF;
    float *sBh = sWh + (J - 1) * HF * HF;
    float *sFi = sBh + (J - 1) * HF;
    float *sWo = sFi + J * 2 * HF;
    float *sBo = sWo + kSynChanChunk * HF;
    float *sWin = sBo + kSynChanChunk;                     // [3][kSynChanChunk]
    const int tid = threadIdx.x, b = blockIdx.y;
    for (int i = tid; i < HF; i += kSynThreads) {
        const bool in = i < H;
        // coefficients of the internal axes (0, 1, 2) = the last N of them carry the grid
        for (int a = 0; a < 3; ++a) {
            const int ua = a - (3 - N);                   // user axis
            sW1[i * 4 + a] = (in && ua >= 0) ? SYN_LD(p.W1, i * N + ua) : 0.f;
        }
        sW1[i * 4 + 3] = in ? SYN_LD(p.b1, i) : 0.f;
        sOm[i] = in ? SYN_LD(p.omega0, i) : 0.f;
        for (int j = 0; j < J; ++j) {
            sFi[(j * 2 + 0) * HF + i] = in ? (p.gamma ? SYN_LD(p.gamma, ((long long)b * J + j) * H + i) : 1.f) : 0.f;
            sFi[(j * 2 + 1) * HF + i] = in ? (p.beta ? SYN_LD(p.beta, ((long long)b * J + j) * H + i) : 0.f) : 0.f;
        }
        for (int j = 0; j + 1 < J; ++j) sBh[j * HF + i] = in ? SYN_LD(p.bh, j * H + i) : 0.f;
    }
    for (int e = tid; e < (J - 1) * HF * HF; e += kSynThreads) {
        const int j = e / (HF * HF), r = (e / HF) % HF, c = e % HF;
        sWh[e] = (r < H && c < H) ? SYN_LD(p.Wh, ((long long)j * H + r) * H + c) : 0.f;
    }
    __syncthreads();
    const long long taps = (long long)p.K[0] * p.K[1] * p.K[2];
    const long long t0 = ((long long)blockIdx.x * kSynThreads + tid) * NC;
    // hidden activations of this thread's taps
    float act[NC][HF];
    float cx[NC][3];
#pragma unroll
    for (int n = 0; n < NC; ++n) {
        long long t = t0 + n;
        if (t >= taps) t = taps - 1;                       // clamped: computed, never stored
        const int m2 = (int)(t % p.K[2]), m1 = (int)((t / p.K[2]) % p.K[1]), m0 = (int)(t / ((long long)p.K[2] * p.K[1]));
        cx[n][0] = axis_coord(m0, p.L[0], p.mode);
        cx[n][1] = axis_coord(m1, p.L[1], p.mode);
        cx[n][2] = axis_coord(m2, p.L[2], p.mode);
    }
#pragma unroll
    for (int i = 0; i < HF; ++i) {
        const float4 w = *reinterpret_cast<const float4 *>(sW1 + 4 * i);
        const float om = sOm[i], ga = sFi[i], be = sFi[HF + i];
#pragma unroll
        for (int n = 0; n < NC; ++n) {
            const float pre = fmaf(w.x, cx[n][0], fmaf(w.y, cx[n][1], fmaf(w.z, cx[n][2], w.w)));
            act[n][i] = fmaf(ga, sin_reduced(om * pre), be);
        }
    }
    for (int j = 1; j < J; ++j) {
        float nxt[NC][HF];
        const float *W = sWh + (j - 1) * HF * HF;
#pragma unroll
        for (int i = 0; i < HF; ++i) {
            float s[NC];
#pragma unroll
            for (int n = 0; n < NC; ++n) s[n] = sBh[(j - 1) * HF + i];
#pragma unroll
            for (int c = 0; c < HF; c += 4) {
                const float4 w = *reinterpret_cast<const float4 *>(W + i * HF + c);
#pragma unroll
                for (int n = 0; n < NC; ++n)
                    s[n] = fmaf(w.x, act[n][c], fmaf(w.y, act[n][c + 1], fmaf(w.z, act[n][c + 2], fmaf(w.w, act[n][c + 3], s[n]))));
            }
            const float ga = sFi[(j * 2) * HF + i], be = sFi[(j * 2 + 1) * HF + i];
#pragma unroll
            for (int n = 0; n < NC; ++n) nxt[n][i] = fmaf(ga, sin_reduced(s[n]), be);
        }
#pragma unroll
        for (int i = 0; i < HF; ++i)
#pragma unroll
            for (int n = 0; n < NC; ++n) act[n][i] = nxt[n][i];
    }
    // output layer and window, a chunk of channels at a time
    T *out = (T *)p.h + (long long)b * p.C * taps;
    for (int c0 = 0; c0 < p.C; c0 += kSynChanChunk) {
        __syncthreads();
        const int nc = p.C - c0 < kSynChanChunk ? p.C - c0 : kSynChanChunk;
        for (int e = tid; e < kSynChanChunk * HF; e += kSynThreads) {
            const int c = e / HF, i = e % HF;
            sWo[e] = (c < nc && i < H) ? SYN_LD(p.Wout, (long long)(c0 + c) * H + i) : 0.f;
        }
        for (int c = tid; c < kSynChanChunk; c += kSynThreads) {
            sBo[c] = c < nc ? SYN_LD(p.bout, c0 + c) : 0.f;
            for (int a = 0; a < 3; ++a) {
                const int ua = a - (3 - N);
                float wv = 0.f;                            // Gaussian: 1 / sigma per axis; causal: alpha in slot 2
                if (c < nc) {
                    if (p.mode == 1) wv = a == 2 ? SYN_LD(p.window, c0 + c) : 0.f;
                    else if (ua >= 0) wv = 1.f / SYN_LD(p.window, (long long)ua * p.C + c0 + c);
                }
                sWin[a * kSynChanChunk + c] = wv;
            }
        }
        __syncthreads();
        for (int c = 0; c < nc; ++c) {
            float s[NC];
#pragma unroll
            for (int n = 0; n < NC; ++n) s[n] = sBo[c];
#pragma unroll
            for (int i = 0; i < HF; i += 4) {
                const float4 w = *reinterpret_cast<const float4 *>(sWo + c * HF + i);
#pragma unroll
                for (int n = 0; n < NC; ++n)
                    s[n] = fmaf(w.x, act[n][i], fmaf(w.y, act[n][i + 1], fmaf(w.z, act[n][i + 2], fmaf(w.w, act[n][i + 3], s[n]))));
            }
            const float w0 = sWin[c], w1 = sWin[kSynChanChunk + c], w2 = sWin[2 * kSynChanChunk + c];
#pragma unroll
            for (int n = 0; n < NC; ++n) {
                float win;
                if (p.mode == 1) win = __expf(-w2 * fabsf(cx[n][2]));
                else {
                    const float a0 = cx[n][0] * w0, a1 = cx[n][1] * w1, a2 = cx[n][2] * w2;
                    win = __expf(-0.5f * (a0 * a0 + a1 * a1 + a2 * a2));
                }
                if (t0 + n < taps) IO<T>::st(out, (long long)(c0 + c) * taps + t0 + n, win * s[n]);
            }
        }
    }
}

// ---- tensor-core version ---------------------------------------------------------------------------------------
// The hidden layers and the output layer are dense contractions: per tile of 128 taps, [128 x HF] activations times
// [HF x HF] (or [HF x 32 channels]) weights.  They run on the tensor cores: one thread issues tcgen05.mma
// (cta_group::1, kind::tf32, M = 128, K = 8 per instruction).  Tap t of a tile is thread t is lane t of tensor memory:
// the activations (the A operand) are written there by their own threads with tcgen05.st, the weights (the B operand)
// sit in shared memory in the K-major layout with the 128-byte swizzle, the accumulator [128 lanes x N columns] sits
// in tensor memory as well, and every thread reads its own tap's row back with tcgen05.ld for the bias, the FiLM
// modulation and the sine, which stay on the ALUs.  (With the activations in shared memory the tensor pipe spent its
// time fetching them: 250 cycles per instruction, 60% of the kernel.)  fp32 accuracy from tf32 products: activations and weights are split x = hi + lo (hi = x rounded
// to tf32, lo = the remainder, of which the tensor cores read the leading tf32 bits) and every contraction is three accumulating products
// hi*hi + hi*lo + lo*hi (the dropped lo*lo term is 2^-22 of the product).  The first layer (N coordinates in, sines of
// arguments of tens of radians) and the window stay in fp32 on the ALUs.  A CTA is persistent over tiles; its weights
// are split and staged once.  The one wait on the tensor cores (mbarrier armed by tcgen05.commit) is bounded: if it
// gives up, the CTA raises the module's status word, stores nothing more and returns.
static __device__ int hn_synth_status;

constexpr int kTcThreads = 128;                          // = taps per tile = rows of the accumulator
constexpr int kTcChan = 32;                              // output channels per contraction

// x rounded to the nearest tf32 (10 explicit mantissa bits) with integer arithmetic: the conversion instruction runs
// on the quarter-rate pipe, which the sines already fill
__device__ __forceinline__ float to_tf32(float x)
{
    return __uint_as_float((__float_as_uint(x) + 0x1000u) & 0xffffe000u);
}

// K-major operand tile in the 128-byte swizzle: a row holds 32 tf32 values of one K block (128 bytes), 8 rows make a
// 1024-byte group, the 16-byte chunk index inside a row is XORed with the row's index in its group, and K blocks
// (columns 32.., for 64 hidden units) follow one another as whole tiles.  Byte offset of element (row, k) of a tile
// of ROWS rows.  (The layout without swizzle, 8 x 16-byte core matrices, puts every row group on the same banks: the
// products then took 200 cycles per instruction and 60% of the kernel's time.)
template <int ROWS> __device__ __forceinline__ int tc_off(int row, int k)
{
    return (k >> 5) * (ROWS * 128) + (row >> 3) * 1024 + (row & 7) * 128 + (((((k & 31) >> 2) ^ (row & 7))) << 4) + (k & 3) * 4;
}

// descriptor of the 8-value K step ks (K block ks / 4) of a tile of ROWS rows, starting at row r0 (a multiple of 8)
template <int ROWS> __device__ __forceinline__ unsigned long long tc_desc(unsigned tile_addr, int ks, int r0 = 0)
{
    const unsigned a = tile_addr + (unsigned)((ks >> 2) * (ROWS * 128) + (r0 >> 3) * 1024 + (ks & 3) * 32);
    return (unsigned long long)((a & 0x3ffffu) >> 4) | (1ull << 16) | ((unsigned long long)(1024 >> 4) << 32) | (1ull << 46) | (2ull << 61);
}

__device__ __forceinline__ void tc_mma_tf32(unsigned tmem_d, unsigned long long da, unsigned long long db, unsigned idesc, unsigned accumulate)
{
    asm volatile("{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
                 " tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, {%5, %6, %7, %8}, p;\n}\n"
                 ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(accumulate), "r"(0u), "r"(0u), "r"(0u), "r"(0u) : "memory");
}
// the same with the A operand in tensor memory ([128 lanes x 8 columns] at ta: row m of the tile is lane m)
__device__ __forceinline__ void tc_mma_tf32_ts(unsigned tmem_d, unsigned ta, unsigned long long db, unsigned idesc, unsigned accumulate)
{
    asm volatile("{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
                 " tcgen05.mma.cta_group::1.kind::tf32 [%0], [%1], %2, %3, {%5, %6, %7, %8}, p;\n}\n"
                 ::"r"(tmem_d), "r"(ta), "l"(db), "r"(idesc), "r"(accumulate), "r"(0u), "r"(0u), "r"(0u), "r"(0u) : "memory");
}
__device__ __forceinline__ void tc_commit(uint64_t *bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n" ::"r"(smem_u32(bar)) : "memory");
}

template <int HF> constexpr size_t synth_tc_smem(int layers)
{
    // weight tiles (per hidden layer [2 HF x HF] = hi rows then lo rows; output chunk [64 x HF]), room to start them
    // on a 1024-byte boundary, small parameters, barrier + tensor-memory slot (the activations live in tensor memory)
    return (size_t)(layers - 1) * 2 * HF * HF * 4 + (size_t)2 * kTcChan * HF * 4 + 1024 +
           sizeof(float) * ((size_t)HF * 4 + HF + (size_t)(layers - 1) * HF + (size_t)layers * 2 * HF + kTcChan + 3 * kTcChan) + 64;
}

template <typename T, int HF>
__global__ void __launch_bounds__(kTcThreads) synth_tc_kernel(SynthArgs p)
{
    extern __shared__ __align__(1024) unsigned char smem_dyn[];
    // the swizzle pattern is a function of the shared-memory address: tiles start on 1024-byte boundaries
    unsigned char *sm = smem_dyn + ((1024u - (smem_u32(smem_dyn) & 1023u)) & 1023u);
    const int J = p.layers, H = p.hidden, N = p.ndim;
    constexpr int TB = 2 * HF * HF * 4, TO = 2 * kTcChan * HF * 4;      // bytes
    unsigned char *sB = sm;                                // [J-1] tiles of [2 HF x HF]: rows 0..HF-1 hi, HF..2HF-1 lo
    unsigned char *sO = sB + (J - 1) * TB;                 // [64 x HF]: rows 0..31 hi, 32..63 lo of the output chunk
    float *sW1 = reinterpret_cast<float *>(sO + TO);
    float *sOm = sW1 + HF * 4;
    float *sBh = sOm + HF;
    float *sFi = sBh + (J - 1) * HF;
    float *sBo = sFi + J * 2 * HF;
    float *sWin = sBo + kTcChan;                           // [3][32]
    uint64_t *bar = reinterpret_cast<uint64_t *>(sWin + 3 * kTcChan);
    unsigned *tslot = reinterpret_cast<unsigned *>(bar + 1);
    const int tid = threadIdx.x, warp = tid >> 5, b = blockIdx.y;
    // tensor memory: accumulator (hi*hi and hi*lo side by side), then this tile's activations, hi and lo: row = lane
    constexpr unsigned DCOLS = 2 * (HF > kTcChan ? HF : kTcChan), TCOLS = DCOLS + 2 * HF;       // 128 or 256 columns
    static_assert((TCOLS & (TCOLS - 1)) == 0 && TCOLS <= 512, "a power of two");
    if (warp == 0) tmem_alloc(smem_u32(tslot), TCOLS);
    if (tid == 0) { mbar_init(bar, 1); fence_mbar_init(); }
    for (int i = tid; i < HF; i += kTcThreads) {
        const bool in = i < H;
        for (int a = 0; a < 3; ++a) {
            const int ua = a - (3 - N);
            sW1[i * 4 + a] = (in && ua >= 0) ? SYN_LD(p.W1, i * N + ua) : 0.f;
        }
        sW1[i * 4 + 3] = in ? SYN_LD(p.b1, i) : 0.f;
        sOm[i] = in ? SYN_LD(p.omega0, i) : 0.f;
        for (int j = 0; j < J; ++j) {
            sFi[(j * 2 + 0) * HF + i] = in ? (p.gamma ? SYN_LD(p.gamma, ((long long)b * J + j) * H + i) : 1.f) : 0.f;
            sFi[(j * 2 + 1) * HF + i] = in ? (p.beta ? SYN_LD(p.beta, ((long long)b * J + j) * H + i) : 0.f) : 0.f;
        }
        for (int j = 0; j + 1 < J; ++j) sBh[j * HF + i] = in ? SYN_LD(p.bh, j * H + i) : 0.f;
    }
    // hidden-layer weights W[out n][in k], split and laid out as the B operand (N rows, K-major)
    for (int e = tid; e < (J - 1) * HF * HF; e += kTcThreads) {
        const int j = e / (HF * HF), n = (e / HF) % HF, k = e % HF;
        const float w = (n < H && k < H) ? SYN_LD(p.Wh, ((long long)j * H + n) * H + k) : 0.f;
        const float hi = to_tf32(w);
        *reinterpret_cast<float *>(sB + j * TB + tc_off<2 * HF>(n, k)) = hi;
        *reinterpret_cast<float *>(sB + j * TB + tc_off<2 * HF>(HF + n, k)) = w - hi;
    }
    fence_async_smem();                                    // generic-proxy writes visible to the tensor cores
    tmem_fence_before_sync();
    __syncthreads();
    tmem_fence_after_sync();
    const unsigned tbase = *tslot;
    const unsigned trow = tmem_addr(tbase, warp, 0);       // this thread's lane, column 0
    const unsigned aB = smem_u32(sB), aO = smem_u32(sO);
    constexpr unsigned IDESC = (1u << 4) | (2u << 7) | (2u << 10) | ((unsigned)(kTcThreads >> 4) << 24);      // f32 out, tf32 in, K-major, M = 128
    auto idesc_n = [](int n) { return IDESC | ((unsigned)(n >> 3) << 17); };
    const long long taps = (long long)p.K[0] * p.K[1] * p.K[2];
    const long long tiles = (taps + kTcThreads - 1) / kTcThreads;
    T *out = (T *)p.h + (long long)b * p.C * taps;
    unsigned phase = 0;
    bool failed = false;
    // One contraction of the activations (in tensor memory) with a weight tile of 2 NB rows (NB hi rows, then NB lo rows):
    // A_hi x [B_hi; B_lo] fills accumulator columns [0, 2 NB) with hi*hi | hi*lo, A_lo x B_hi adds lo*hi to columns
    // [0, NB): 2 * HF / 8 instructions.  The caller adds the two halves when it reads its row.
    auto contract = [&](unsigned ab, auto nb_tag) {
        constexpr int NB = decltype(nb_tag)::value;
        if (tid == 0) {
            tmem_fence_after_sync();
#pragma unroll
            for (int ks = 0; ks < HF / 8; ++ks)
                tc_mma_tf32_ts(tbase, tbase + DCOLS + ks * 8, tc_desc<2 * NB>(ab, ks), idesc_n(2 * NB), ks != 0);
#pragma unroll
            for (int ks = 0; ks < HF / 8; ++ks)
                tc_mma_tf32_ts(tbase, tbase + DCOLS + HF + ks * 8, tc_desc<2 * NB>(ab, ks), idesc_n(NB), 1);
            tc_commit(bar);
        }
        const bool ok = mbar_wait(bar, phase);
        failed = __syncthreads_or(!ok) != 0;                // one decision for the whole CTA
        phase ^= 1u;
        tmem_fence_after_sync();
    };
    // this thread's activations -> its lane of the A operand in tensor memory, split
    auto put_acts = [&](const float (&act)[HF]) {
#pragma unroll
        for (int c0 = 0; c0 < HF; c0 += 16) {
            float hi[16], lo[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                hi[i] = to_tf32(act[c0 + i]);
                lo[i] = act[c0 + i] - hi[i];               // the tensor cores read its leading tf32 bits (2^-11 of 2^-11 is dropped)
            }
            TmemIO<16>::st(trow + DCOLS + c0, hi);
            TmemIO<16>::st(trow + DCOLS + HF + c0, lo);
        }
        tmem_wait_st();
        tmem_fence_before_sync();                          // (this thread's tensor-memory reads and writes precede the next product)
        __syncthreads();
    };
    for (long long tile = blockIdx.x; tile < tiles && !failed; tile += gridDim.x) {
        long long t = tile * kTcThreads + tid;
        const bool live = t < taps;
        if (!live) t = taps - 1;                           // clamped: computed, never stored
        const int m2 = (int)(t % p.K[2]), m1 = (int)((t / p.K[2]) % p.K[1]), m0 = (int)(t / ((long long)p.K[2] * p.K[1]));
        const float cx0 = axis_coord(m0, p.L[0], p.mode), cx1 = axis_coord(m1, p.L[1], p.mode), cx2 = axis_coord(m2, p.L[2], p.mode);
        float act[HF];
#pragma unroll
        for (int i = 0; i < HF; ++i) {
            const float4 w = *reinterpret_cast<const float4 *>(sW1 + 4 * i);
            const float pre = fmaf(w.x, cx0, fmaf(w.y, cx1, fmaf(w.z, cx2, w.w)));
            act[i] = fmaf(sFi[i], sin_reduced(sOm[i] * pre), sFi[HF + i]);
        }
        for (int j = 1; j < J; ++j) {
            put_acts(act);
            contract(aB + (j - 1) * TB, std::integral_constant<int, HF>{});
            if (failed) break;
#pragma unroll
            for (int c0 = 0; c0 < HF; c0 += 16) {
                float acc[16], acl[16];
                TmemIO<16>::ld(acc, trow + c0);
                TmemIO<16>::ld(acl, trow + HF + c0);
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 16; ++i)
                    act[c0 + i] = fmaf(sFi[(j * 2) * HF + c0 + i], sin_reduced((acc[i] + acl[i]) + sBh[(j - 1) * HF + c0 + i]), sFi[(j * 2 + 1) * HF + c0 + i]);
            }
        }
        if (failed) break;
        put_acts(act);                                      // operand of every output chunk
        for (int c0 = 0; c0 < p.C; c0 += kTcChan) {
            const int nc = p.C - c0 < kTcChan ? p.C - c0 : kTcChan;
            // output weights of this chunk (one chunk: staged once per CTA; more: once per tile and chunk)
            if (tile == (long long)blockIdx.x || p.C > kTcChan) {
                for (int e = tid; e < kTcChan * HF; e += kTcThreads) {
                    const int c = e / HF, k = e % HF;
                    const float w = (c < nc && k < H) ? SYN_LD(p.Wout, (long long)(c0 + c) * H + k) : 0.f;
                    const float hi = to_tf32(w);
                    *reinterpret_cast<float *>(sO + tc_off<2 * kTcChan>(c, k)) = hi;
                    *reinterpret_cast<float *>(sO + tc_off<2 * kTcChan>(kTcChan + c, k)) = w - hi;
                }
                for (int c = tid; c < kTcChan; c += kTcThreads) {
                    sBo[c] = c < nc ? SYN_LD(p.bout, c0 + c) : 0.f;
                    for (int a = 0; a < 3; ++a) {
                        const int ua = a - (3 - N);
                        float wv = 0.f;                    // Gaussian: 1 / sigma per axis; causal: alpha in slot 2
                        if (c < nc) {
                            if (p.mode == 1) wv = a == 2 ? SYN_LD(p.window, c0 + c) : 0.f;
                            else if (ua >= 0) wv = 1.f / SYN_LD(p.window, (long long)ua * p.C + c0 + c);
                        }
                        sWin[a * kTcChan + c] = wv;
                    }
                }
                fence_async_smem();
                tmem_fence_before_sync();
                __syncthreads();
            }
            contract(aO, std::integral_constant<int, kTcChan>{});
            if (failed) break;
#pragma unroll
            for (int q0 = 0; q0 < kTcChan; q0 += 16) {
                float acc[16], acl[16];
                TmemIO<16>::ld(acc, trow + q0);
                TmemIO<16>::ld(acl, trow + kTcChan + q0);
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 16; ++i) acc[i] += acl[i];
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const int c = q0 + i;
                    float win;
                    if (p.mode == 1) win = __expf(-sWin[2 * kTcChan + c] * fabsf(cx2));
                    else {
                        const float a0 = cx0 * sWin[c], a1 = cx1 * sWin[kTcChan + c], a2 = cx2 * sWin[2 * kTcChan + c];
                        win = __expf(-0.5f * (a0 * a0 + a1 * a1 + a2 * a2));
                    }
                    if (live && c < nc) IO<T>::st(out, (long long)(c0 + c) * taps + t, win * (acc[i] + sBo[c]));
                }
            }
            if (p.C > kTcChan) {
                // the next chunk's weights overwrite sO and the next product overwrites the accumulator
                tmem_fence_before_sync();
                __syncthreads();
            }
        }
    }
    if (failed) atomicExch(&hn_synth_status, 1);
    tmem_fence_before_sync();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tbase, TCOLS);
}

int synth_device_status()
{
    int v = 0;
    if (cudaDeviceSynchronize() != cudaSuccess) return -1;
    if (cudaMemcpyFromSymbol(&v, hn_synth_status, sizeof(int)) != cudaSuccess) return -1;
    return v;
}

template <typename T, int HF> static int launch_synth_tc_t(const SynthArgs &a, cudaStream_t st)
{
    const long long taps = (long long)a.K[0] * a.K[1] * a.K[2];
    const long long tiles = (taps + kTcThreads - 1) / kTcThreads;
    const size_t sm = synth_tc_smem<HF>(a.layers);
    if (tiles <= 0 || a.B > 65535 || sm > 160 * 1024) return -1;
    static int sms = 0;
    if (!sms) {
        int dev = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (sms <= 0) sms = 148;
    }
    static DevOnce attr;
    if (attr.first()) cudaFuncSetAttribute(synth_tc_kernel<T, HF>, cudaFuncAttributeMaxDynamicSharedMemorySize, 160 * 1024);
    // persistent CTAs: as many as fit (shared memory, 512 tensor-memory columns per SM), at most one per tile
    long long per_sm = (220 * 1024) / (long long)(sm + 1024);
    const long long by_tmem = 512 / (2 * (HF > kTcChan ? HF : kTcChan) + 2 * HF);
    if (per_sm > by_tmem) per_sm = by_tmem;
    if (per_sm > 8) per_sm = 8;
    if (per_sm < 1) per_sm = 1;
    long long grid = (long long)sms * per_sm / (a.B < sms * per_sm ? a.B : 1);
    if (grid < 1) grid = 1;
    if (grid > tiles) grid = tiles;
    synth_tc_kernel<T, HF><<<dim3((unsigned)grid, (unsigned)a.B), kTcThreads, sm, st>>>(a);
    return 1;
}

bool synth_supported(int hidden, int layers) { return hidden >= 1 && hidden <= 64 && layers >= 1 && layers <= 8; }

template <typename T, int HF, int NC> static int launch_synth_t(const SynthArgs &a, cudaStream_t st)
{
    const long long taps = (long long)a.K[0] * a.K[1] * a.K[2];
    const long long per_block = (long long)kSynThreads * NC;
    const long long blocks = (taps + per_block - 1) / per_block;
    if (blocks <= 0 || blocks > 0x7fffffffll || a.B > 65535) return -1;
    const size_t sm = sizeof(float) * ((size_t)HF * 4 + HF + (size_t)(a.layers - 1) * HF * HF + (size_t)(a.layers - 1) * HF +
                                       (size_t)a.layers * 2 * HF + (size_t)kSynChanChunk * HF + kSynChanChunk + 3 * kSynChanChunk);
    if (sm > 200 * 1024) return -1;
    static DevOnce attr;
    if (attr.first()) cudaFuncSetAttribute(synth_kernel<T, HF, NC>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    synth_kernel<T, HF, NC><<<dim3((unsigned)blocks, (unsigned)a.B), kSynThreads, sm, st>>>(a);
    return 1;
}

int launch_synth(const SynthArgs &a, cudaStream_t st)
{
    if (!synth_supported(a.hidden, a.layers)) return -1;
    // tensor-core version for 17 .. 64 hidden units wherever its operands fit in shared memory (else the ALU version)
    if (!a.no_tensor_cores) {
        int n = -1;
        if (a.hidden <= 16) n = -1;                        // 16 units: the products are too small to pay for the round trips
        else if (a.hidden <= 32) n = a.dtype == 0 ? launch_synth_tc_t<float, 32>(a, st) : launch_synth_tc_t<bf16, 32>(a, st);
        else n = a.dtype == 0 ? launch_synth_tc_t<float, 64>(a, st) : launch_synth_tc_t<bf16, 64>(a, st);
        if (n >= 0) return n;
    }
#define HN_SYN(T)                                                                   \
    do {                                                                            \
        if (a.hidden <= 16) return launch_synth_t<T, 16, 2>(a, st);                 \
        if (a.hidden <= 32) return launch_synth_t<T, 32, 2>(a, st);                 \
        return launch_synth_t<T, 64, 1>(a, st);                                     \
    } while (0)
    if (a.dtype == 0) HN_SYN(float);
    HN_SYN(bf16);
#undef HN_SYN
}

}  // namespace hn
