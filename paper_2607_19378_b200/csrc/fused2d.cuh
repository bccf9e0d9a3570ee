// Fused 2-D kernel (fused2d.cu): interface used by the scheduler.
#pragma once
#include <cuda_runtime.h>

namespace hn {

struct Fused2dArgs {
    const void *q, *k, *v, *h;
    void *y;
    const void *q2;           // optional second gate and result of the same convolution: y2 = q2 * (h conv (k v)); both or none
    void *y2;
    long long slices;         // B*C
    int lx, ly;               // grid extent along x (contiguous) and y
    long long h_mod, h_off;   // filter slice = h_mod ? (s + h_off) % h_mod : s
    float scale;              // 1 / (P*P)
    const float2 *gtw;        // global twiddle table with gtw_n >= P points
    int gtw_n;
    long long kv_elems, h_elems;   // total elements of k (= v) and of h: bounds for aligned row fetches
};

bool fused2d_supported(int log2p);
int launch_fused2d(const Fused2dArgs &a, int log2p, int dtype, cudaStream_t st);

}  // namespace hn
