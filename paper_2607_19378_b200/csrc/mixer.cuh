// Pointwise stages of the full HyenaND operator (Eq. 2 of the paper) around the long convolution (mixer.cu).
#pragma once
#include <cuda_runtime.h>

namespace hn {

// q, k, v: [nb][C][L] in the I/O dtype (0 = fp32, 1 = bf16).  Writes, in fp32 and the same layout,
//   kz = l2(q) * g_in * rsqrt(mean_c((l2(q) SiLU(k))^2) + eps)    (first factor of the inner gate)
//   vz = SiLU(k)                                                  (second factor)
//   qz = Sigmoid(v)                                               (outer gate)
// so that the long convolution called on (qz, kz, vz) returns Sigmoid(v) * (K conv RMSNorm(l2(q) SiLU(k))).
int launch_mixer_pre(const void *q, const void *k, const void *v, const float *g_in, float eps, int dtype,
                     long long nb, int C, long long L, float *qz, float *kz, float *vz, cudaStream_t st);
// o: [nb][C][L] fp32 (the gated convolution); y = RMSNorm over the channels of each token, weight g_out, in the I/O dtype
int launch_mixer_post(const float *o, const float *g_out, float eps, int dtype, long long nb, int C, long long L,
                      void *y, cudaStream_t st);
// widen n elements of the I/O dtype to fp32 (the kernel h of a bf16 problem)
int launch_widen(const void *src, int dtype, long long n, float *dst, cudaStream_t st);

}  // namespace hn
