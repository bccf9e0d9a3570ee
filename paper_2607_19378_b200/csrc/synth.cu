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

namespace hn {

// parameter loads (checked in the checked build)
#define SYN_LD(ptr, idx) (HN_G((ptr) + (idx), 4), (ptr)[idx])

constexpr int kSynThreads = 128;
constexpr int kSynChanChunk = 32;        // output channels whose weights sit in shared memory at a time

__device__ __forceinline__ float sin_reduced(float x)
{
    const float k = rintf(x * 0.15915494309189535f);
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
