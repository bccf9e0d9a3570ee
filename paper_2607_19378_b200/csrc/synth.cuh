// Kernel synthesis (synth.cu): K(x) = window * SIREN(coordinates; FiLM) written in the layout the convolution reads.
#pragma once
#include <cuda_runtime.h>

namespace hn {

struct SynthArgs {
    int ndim, mode;           // mode: 0 linear (2L-1 taps per axis), 1 causal, 2 circular
    int L[3], K[3];           // grid and tap extents, leading axes of extent 1 (internal 3-axis form)
    int B, C, hidden, layers;
    const float *W1, *b1, *omega0;     // [hidden][ndim], [hidden], [hidden]
    const float *Wh, *bh;              // [layers-1][hidden][hidden], [layers-1][hidden]
    const float *Wout, *bout;          // [C][hidden], [C]
    const float *gamma, *beta;         // [B][layers][hidden] or NULL (identity modulation)
    const float *window;               // Gaussian: sigma [ndim][C]; causal: alpha [C]
    void *h;                           // [B][C][K...] in the I/O dtype
    int dtype;
    int no_tensor_cores;               // 1: the ALU version (development switch HYENAND_SYNTH_ALU)
};

bool synth_supported(int hidden, int layers);
int launch_synth(const SynthArgs &a, cudaStream_t st);
// 0, or 1 once a bounded wait on the tensor cores has given up (synchronises the device); -1 if it cannot be read
int synth_device_status();

}  // namespace hn
