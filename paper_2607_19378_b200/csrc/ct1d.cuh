// Long 1-D path (padded length above the shared-memory line limit): the
// transform is split Cooley-Tukey style into two passes over a 2-D view of the
// sequence (Appendix B.3 of the paper describes the same decomposition).
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>

#include "common.cuh"

namespace hn {

struct Ct1dPlan {
    int L, K, log2p, B, C, causal, dtype;
    int log2p1, log2p2;       // P = P1 * P2, n = n1*P2 + n2, k = k1 + P1*k2
    float2 *wu;               // [slices_per_chunk][P1/2+1][P2]
    float2 *wh;               // [C or slices_per_chunk][P1/2+1][P2]
    float2 *tw1, *tw2;        // twiddle tables for P1 and P2
    float2 *twp_coarse, *twp_fine;   // W_P^j = coarse[j >> lo] * fine[j & (2^lo - 1)]
    int lo;
    int *status;              // device word set when a bounded wait on a tensor copy gives up (owned by the plan)
    Switches sw;              // development switches, read when the plan was created
    long long slices_per_chunk, wh_slices;
    long long r0, r1;         // slices [r0, r1) the next forward works on
    int dt_in, dt_out, dt_h;  // element types of k and v, of the gate q and the result y, of the taps h for the next forward
                              // (all equal to dtype unless the caller of ct1d_forward sets them: every stage takes its
                              // element type per launch)
    int keep_filter;          // 1: the spectrum of the shared filter is still in wh from this plan's previous forward
                              // (same taps): the next forward does not transform it again
};

// allocations go on the plan's guarded list `g` and are freed with it
int ct1d_init(Ct1dPlan *c, int L, int K, int log2p, int B, int C, int causal, int dtype, const Switches &sw,
              GuardedAllocs *g, size_t *bytes);
int ct1d_forward(Ct1dPlan *c, const void *q, const void *k, const void *v, const void *h, bool shared,
                 void *y, cudaStream_t st, int *launches, Prof *prof);
int ct1d_launches(const Ct1dPlan *c, bool shared);
bool ct1d_uses_w(const Ct1dPlan *c);
// true when a forward of this plan may read/write tensors of element type `dtype` (0: fp32, else bf16) in any stage
bool ct1d_takes_dtype(const Ct1dPlan *c, int dtype);

// warp-engine kernels (ct1d_w.cu)
bool ct1d_w_supported(int log2p1, int log2p2, int L, int K, int causal, int dtype);
int ct1d_w_filter(Ct1dPlan *c, const void *h, long long n, bool staged_ok, cudaStream_t st, int *launches, Prof *prof,
                  int (*fallback)(Ct1dPlan *, const char *, long long, cudaStream_t, int *, Prof *));
int ct1d_w_body(Ct1dPlan *c, const void *q, const void *k, const void *v, long long n, bool shared, long long s0,
                void *y, cudaStream_t st, int *launches, Prof *prof);

}  // namespace hn
