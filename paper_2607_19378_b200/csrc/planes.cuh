// Plane-fused kernels (planes.cu): interface used by the scheduler.
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>

namespace hn {

enum PlaneKind { PLANE_U = 0, PLANE_H = 1, PLANE_INV = 2 };

struct PlaneArgs {
    const void *a;        // k (PLANE_U), h (PLANE_H), q (PLANE_INV; NULL: no gate, the convolution itself is written)
    const void *b;        // v (PLANE_U)
    float2 *out;          // spectra [plane][P/2+1][P] written by PLANE_U / PLANE_H
    const float2 *in;     // spectra read by PLANE_INV
    void *y;              // output of PLANE_INV
    const void *q2;       // PLANE_INV: optional second gate and result of the same planes, y2 = q2 * planes (both or none)
    void *y2;
    long long planes;     // number of x-y planes
    int lx, ly;           // grid extent along x (contiguous) and y
    const float2 *gtw;    // global twiddle table with gtw_n >= P points
    int gtw_n;
    long long a_elems;    // total elements of a (and b): bounds for the aligned row fetches
};

bool plane_supported(int log2p);
int launch_plane(const PlaneArgs &a, int which, int log2p, int dtype, cudaStream_t st);

}  // namespace hn
