// Spectral core with TMA tile copies (core_tma.cu): interface used by the scheduler.
#pragma once
#include <cuda_runtime.h>
#include "common.cuh"

namespace hn {

// Tensor maps of the two fixed workspace buffers the core reads (k*v spectra, also written back in
// place; filter spectra), plus what they were built for, so a launch can check it matches.
struct CoreTmaMaps {
    alignas(64) unsigned char u[128];
    alignas(64) unsigned char h[128];
    const float2 *in, *h_base;
    int nc, n_in, h_n_in, log2p;
    long long in_outer, h_outer, max_outer, h_outer_count;
    bool valid;
};

// true if `a` is a case the TMA core handles (256- or 1024-point axis, in place, even number of bins) and the
// driver offers tensor-map encoding
bool core_tma_supported(const AxisArgs &a);
// builds the maps for buffers a.in (max_outer outer entries) and a.h (h_outer_count entries)
bool core_tma_make(CoreTmaMaps *m, const AxisArgs &a, long long max_outer, long long h_outer_count);
// launches on `st`; -1 if the arguments do not match the maps (nothing launched); *status (device
// word) is set non-zero by the kernel if a bounded wait on a copy gave up
int launch_core_tma(const AxisArgs &a, const CoreTmaMaps &m, int *status, cudaStream_t st);

}  // namespace hn
