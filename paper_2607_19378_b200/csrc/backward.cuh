// Index-remapping and pointwise helpers of the backward pass (backward.cu).
#pragma once
#include <cuda_runtime.h>

namespace hn {

// How the source index along one axis follows from the output index i (G = output extent, Ls = source extent):
enum RemapMode {
    REMAP_PAD = 0,      // j = i                       (zero-padding: entries with j >= Ls are zero)
    REMAP_NEG = 1,      // j = (G - i) mod G           (the opposite displacement on a ring of G points)
    REMAP_REV = 2,      // j = Ls - 1 - i              (reversal; zero where j falls outside the source)
    REMAP_WRAP = 3      // j = (i - shift) mod Ls      (taps read back from a padded ring: displacement i - shift)
};

struct RemapArgs {
    const float *a, *b;       // sources [slices][Ls0][Ls1][Ls2]; b may be NULL (no product)
    float *out;               // [slices][G0][G1][G2]
    long long slices;
    int G[3], Ls[3], mode[3], shift[3];
    int a_bf16, out_bf16;     // the sources (a, and b when there is one) and/or out hold bf16 instead of fp32
};

// out[s][i] = a[s][j(i)] * (b ? b[s][j(i)] : 1), zero where an axis index falls outside the source
int launch_remap(const RemapArgs &r, cudaStream_t st);
int launch_fill(float *dst, float value, long long n, cudaStream_t st);
// dst (I/O dtype) = a * (b ? b : 1); b holds elements of b_dtype (0: fp32, else bf16)
int launch_mul_cast(const float *a, const void *b, int b_dtype, long long n, int dtype, void *dst, cudaStream_t st);
// acc[c][t] (+)= sum over nb of src[(b * C + c)][t]   (set = true overwrites)
int launch_batch_sum(const float *src, long long nb, long long C, long long kvol, bool set, float *acc, cudaStream_t st);

}  // namespace hn
