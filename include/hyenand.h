/*
 * hyenand.h -- C ABI of the B200 (sm_100a) gated N-D long convolution.
 *
 * The library computes, for every batch entry b, channel c and grid position i
 * of a 1-D, 2-D or 3-D grid L_1 x ... x L_N,
 *
 *     y[b,c,i] = q[b,c,i] * sum_j h[b,c, i - j] * k[b,c,j] * v[b,c,j]
 *
 * i.e. the gated Hyena mixer (Definition A.3; Eq. 1-2 without the pointwise
 * activations and norms, which the caller applies to q, k, v beforehand): k*v is
 * the inner gate, h the depthwise long-convolution kernel whose weight depends
 * on the displacement i - j only (Definition A.2, Theorem A.5), q the outer
 * gate.  The sum is evaluated through FFTs on the zero-padded grid (Section
 * 3.2.1 "non-circular convolutions", Appendix B.1 Eq. 11-13): pad each axis to
 * P_n >= 2 L_n - 1 (a power of two), transform k*v and h, multiply the
 * spectra, transform back, crop, apply q.  All arithmetic is fp32; bf16 is an
 * I/O format only (one round-to-nearest-even at the final store).
 *
 * Layout (all buffers dense, row-major, last axis contiguous):
 *     q, k, v, y : [B][C][L_1]...[L_N]
 *     h          : [B][C][K_1]...[K_N]
 *       non-causal: K_n = 2 L_n - 1, tap index m_n = (i_n - j_n) + (L_n - 1)
 *       causal (N = 1 only, Appendix A.3 masking strategy): K_1 = L_1, tap
 *       index m = i - j >= 0, negative displacements have weight zero.
 *     One dtype for all five buffers.
 *
 * Ownership: the caller owns q, k, v, h, y.  A plan owns its device workspace
 * and twiddle tables.  hyenand_forward* never allocates device memory, never
 * synchronises and only enqueues work on the given stream (hyenand_forward_host
 * is the exception, see below).  One forward may be in flight per plan; use one
 * plan per concurrent stream.  Plans belong to the device that was current
 * when they were created.
 *
 * Errors: functions returning int return HYENAND_OK or an error code and
 * record a message for hyenand_last_error() (thread-local).  On error nothing
 * is launched.  NaN/Inf in an input spreads to its whole (b,c) slice; that is
 * not an error.
 */
#ifndef HYENAND_H
#define HYENAND_H

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct hyenand_plan hyenand_plan;   /* opaque, library-owned */

enum { HYENAND_F32 = 0, HYENAND_BF16 = 1 };

enum {
    HYENAND_OK = 0,
    HYENAND_ERR_INVALID_ARG = 1,   /* bad count, null or misaligned pointer, aliasing */
    HYENAND_ERR_UNSUPPORTED = 2,   /* causal with ndim > 1, axis too long */
    HYENAND_ERR_ALLOC = 3,         /* workspace could not be allocated */
    HYENAND_ERR_CUDA = 4           /* a CUDA call or launch failed */
};

/*
 * Create a plan for grids dims[0..ndim-1] (host array), batch B, C channels.
 * ndim in {1,2,3}; every L_n >= 1; causal in {0,1} (1 requires ndim == 1);
 * dtype HYENAND_F32 or HYENAND_BF16.  Allocates the workspace and twiddle
 * tables on the current device (this call may synchronise).  Returns NULL on
 * failure, reason in hyenand_last_error().
 * Limits: for ndim >= 2 each padded axis P_n <= 8192; for ndim == 1,
 * P_1 <= 2^24 (L_1 <= 8388608; the parity tests run up to that length).
 */
hyenand_plan *hyenand_create_plan(int ndim, const int *dims, int B, int C, int causal, int dtype);

/*
 * Same with the boundary handling named explicitly (Section 3.2.1, circular and non-circular convolutions):
 *   HYENAND_MODE_LINEAR    zero-padded, non-causal: the kernel lives on (2 L_1 - 1) x ... x (2 L_N - 1)
 *   HYENAND_MODE_CAUSAL    1-D only (Appendix A.3): K_1 = L_1, negative displacements carry no weight
 *   HYENAND_MODE_CIRCULAR  periodic boundaries: the kernel lives on the grid itself, K_n = L_n, tap index
 *                          m_n = (i_n - j_n) mod L_n, and the transforms run on L_n points with no padding.
 *                          Every L_n must be a power of two and at most 8192 (HYENAND_ERR_UNSUPPORTED otherwise).
 * hyenand_create_plan(..., causal, ...) is this call with mode = causal ? CAUSAL : LINEAR.
 */
enum { HYENAND_MODE_LINEAR = 0, HYENAND_MODE_CAUSAL = 1, HYENAND_MODE_CIRCULAR = 2 };
hyenand_plan *hyenand_create_plan_mode(int ndim, const int *dims, int B, int C, int mode, int dtype);

/*
 * One forward pass with one filter per (b,c): the input-dependent kernels of
 * Section 3.2.2, one per sample of the batch and per channel.
 * q, k, v, h, y: DEVICE pointers, 16-byte aligned, y must not alias an input.
 * cuda_stream: a cudaStream_t (NULL = the legacy default stream).
 */
int hyenand_forward(hyenand_plan *plan, const void *q, const void *k, const void *v,
                    const void *h, void *y, void *cuda_stream);

/*
 * Same with an explicit batch stride for h, in elements: 0 means h is
 * [C][K_1]..[K_N], one kernel per channel shared by the whole batch (the
 * static kernel of Section 3.2.1); C*K_1*..*K_N is the dense per-sample layout.
 * Other values are rejected.
 */
int hyenand_forward_ex(hyenand_plan *plan, const void *q, const void *k, const void *v,
                       const void *h, long long h_batch_stride_elems, void *y, void *cuda_stream);

/*
 * End-to-end variant: q, k, v, h, y are HOST pointers (pinned memory gives the
 * fastest copies and is needed for the copies to overlap; any host memory
 * works).  Copies the inputs to device staging buffers owned by the plan
 * (allocated on the first call, which therefore may synchronise), runs the
 * same kernels as hyenand_forward_ex and copies y back.  Problems above 64 MB
 * are pipelined over up to eight groups of (b,c) slices: the inputs of the next
 * group travel on a copy stream of the plan while the current group is computed
 * on cuda_stream and the previous group's result travels back on a second copy
 * stream (a filter shared over the batch is copied first, whole).  The copy
 * streams start after the work already queued on cuda_stream.  The result is
 * bit-identical to hyenand_forward_ex on device copies of the same tensors.
 * Returns after y has arrived on the host (the call synchronises all three
 * streams).
 */
int hyenand_forward_host(hyenand_plan *plan, const void *q, const void *k, const void *v,
                         const void *h, long long h_batch_stride_elems, void *y, void *cuda_stream);

/* Frees the workspace (synchronises the device).  NULL is accepted. */
void hyenand_destroy_plan(hyenand_plan *plan);

/* Message of the last error on this thread ("" if none).  Never NULL. */
const char *hyenand_last_error(void);

/* Code of the last error on this thread (HYENAND_OK if the last call succeeded);
 * tells why hyenand_create_plan returned NULL. */
int hyenand_last_error_code(void);

/* Device-side status of the plan's kernels.  Every wait a kernel makes on an asynchronous copy is
 * bounded; a kernel whose wait gave up writes a non-zero code here and returns instead of hanging.
 * Reads that word back (a blocking device-to-host copy of 4 bytes: call it after synchronising the
 * stream).  Returns 0 if no kernel reported anything, the code otherwise, -1 on error.  The paper has
 * no counterpart; it exists so that a failed copy is observable from the host. */
int hyenand_plan_device_status(hyenand_plan *plan);

/* Guard bands.  Every device allocation of a plan (workspace sets, twiddle tables, status word) sits between two
 * bands of 4096 bytes filled with a fixed byte when the plan is created.  Returns how many of those bytes no
 * longer hold it, i.e. 0 unless a kernel wrote outside the plan's workspace; -1 on error.  Blocking (copies the
 * bands to the host): call it after synchronising the stream.  The paper has no counterpart; it stands in for a
 * memory checker on machines where none can be run. */
long long hyenand_plan_guard_damage(hyenand_plan *plan);

/* Checked build.  libhyenand_debug.so is this library compiled with -DHYENAND_DEBUG: every load, store, asynchronous
 * copy and L2 prefetch a kernel makes to global memory is first compared with the address ranges the call may touch
 * (the caller's tensors and the device allocations of the objects involved; tensor copies are bounded by their
 * tensor maps and shared-memory indices are not checked).  An access outside all ranges is counted; it is still made.
 * hyenand_debug_build returns 1 in that library, 0 in the product library.  hyenand_debug_violations synchronises the
 * device and returns the number of such accesses since the last call (clearing the count), with the address, source
 * line and source file of the first one; -1 in the product library.  The paper has no counterpart; it stands in for
 * a memory checker on machines where none can be run.  Every call of the checked library synchronises the device. */
int hyenand_debug_build(void);
long long hyenand_debug_violations(unsigned long long *first_address, int *first_line, const char **file);
/* Self-test of the checked build: fills a registered and an unregistered device buffer of 1000 floats (both valid
 * allocations, so nothing faults) and returns the number of accesses the checker counted for the second one
 * (1000 when it works); -1 in the product library, -2 when memory could not be had, -3 when the registered buffer
 * was flagged, -4 when the reported address lies outside the unregistered buffer. */
long long hyenand_debug_selftest(void);

/* Self-test of the mechanism behind hyenand_plan_device_status: launches one small CTA that waits, for at
 * most `polls` polls (clamped to [1, 65536]), on a barrier that nothing ever completes.  The wait must run out
 * and the kernel must report it: returns 9 (the code that kernel records), 0 if the wait wrongly succeeded,
 * -1 on a CUDA error.  Blocking; allocates and frees 4 bytes of device memory.  No counterpart in the paper. */
int hyenand_selftest_bounded_wait(int polls);

/* Reporting helpers (host-only, no device work). */
size_t hyenand_plan_workspace_bytes(const hyenand_plan *plan);        /* device bytes owned by the plan: workspace, plus the
                                                                       * staging copies once hyenand_forward_host has run, plus
                                                                       * room for C filter spectra once a filter shared over the
                                                                       * batch has been used (allocated by that first call) */
int hyenand_plan_fft_dims(const hyenand_plan *plan, int *out_P);      /* writes ndim padded sizes P_n */
int hyenand_plan_launches(const hyenand_plan *plan, int h_shared);    /* kernels enqueued by one forward */
const char *hyenand_plan_path(const hyenand_plan *plan);              /* name of the kernel path chosen */
/* How the batch is scheduled: slices per group and the number of lanes (workspace sets with a stream each; 1 =
 * everything on the caller's stream).  Either pointer may be NULL. */
int hyenand_plan_groups(const hyenand_plan *plan, long long *slices_per_group, int *lanes);


/*
 * The full HyenaND operator, Eq. 2 (Section 3.2):
 *
 *     y = RMSNorm_out( Sigmoid(v) * ( K conv RMSNorm_in( l2(q) * SiLU(k) ) ) )
 *
 * q, k, v are the projected inputs [B][C][L_1]..[L_N], h the kernel K laid out as for hyenand_forward_ex, g_in and
 * g_out the C fp32 weights of the two RMSNorms (device pointers).  l2 and both RMSNorms act per token (one grid
 * position of one batch entry) across the C channels: l2(q) = q / max(||q||_2, 1e-12); RMSNorm(x) = x /
 * sqrt(mean_c(x^2) + eps) * g, eps as given at creation (>= 0).  The pointwise stages are kernels of their own before
 * and after the long convolution; everything between the first read of q, k, v and the store of y stays fp32 (the
 * convolution runs on an fp32 plan even when the I/O type is bf16; the taps h are read in the caller's type where the
 * path transforms the filter in kernels of its own, and widened once per call elsewhere), so y carries one rounding.  mode: HYENAND_MODE_*.  The object owns an fp32 plan and fp32 scratch for at most 2 GiB worth of batch
 * entries per pass; hyenand_mixer_plan exposes the inner plan for the reporting helpers (do not destroy it).
 * Errors and stream semantics as hyenand_forward_ex.  hyenand_mixer_guard_damage: as hyenand_plan_guard_damage, over
 * the scratch and the inner plan.
 */
typedef struct hyenand_mixer hyenand_mixer;
hyenand_mixer *hyenand_mixer_create(int ndim, const int *dims, int B, int C, int mode, int dtype, float eps);
int hyenand_mixer_forward(hyenand_mixer *mixer, const void *q, const void *k, const void *v, const void *h,
                          long long h_batch_stride_elems, const float *g_in, const float *g_out, void *y,
                          void *cuda_stream);
hyenand_plan *hyenand_mixer_plan(hyenand_mixer *mixer);
long long hyenand_mixer_guard_damage(hyenand_mixer *mixer);
void hyenand_mixer_destroy(hyenand_mixer *mixer);

/*
 * Backward pass of the gated long convolution (the paper defines and benchmarks the forward only, Appendix B.4;
 * this is the derivative of Definition A.3).  With y = q * (h conv (k v)) and dy given:
 *     dq = dy * (h conv (k v));   du = h' conv (dy q) with h'[d] = h[-d];   dk = du * v;   dv = du * k;
 *     dh[d] = sum_i (dy q)_i (k v)_{i-d} for every displacement d that has a tap, summed over the batch as well when
 *     the kernel is shared (h_batch_stride_elems = 0; dh then has the shape of h, [C][K..]).
 * q, k, v, dy, dq, dk, dv: [B][C][L..]; h, dh: as hyenand_forward_ex; all DEVICE pointers of the one I/O dtype,
 * 16-byte aligned; no output may overlap an input or another output (checked: HYENAND_ERR_INVALID_ARG, nothing is
 * launched).  Every gradient is accumulated in fp32 and rounded once, at its store.  The gradients are long
 * convolutions themselves and run on the forward's kernels: dq is a forward gated by dy; du is a forward of dy q against
 * the kernel at the opposite displacement, leaving through the two gates v and k as dk and dv where the path's last
 * kernel takes a second gate (else through an fp32 du); dh is the full linear convolution of dy q with the reversed
 * k v on the general N-D kernels (circular mode: one circular convolution; 1-D grids whose padded length exceeds 8192:
 * one or two causal convolutions of reversed signals).  With bf16 I/O the kernels read the caller's tensors themselves
 * wherever the path takes an element type per launch; elsewhere the inputs are widened once.
 * The handle owns up to three plans and the scratch (about 4 GiB for the batch groups, 2 GiB for the dh groups).
 * Limits: as the forward's; circular mode needs power-of-two grids.  Errors and stream semantics as hyenand_forward_ex.
 */
typedef struct hyenand_grad hyenand_grad;
hyenand_grad *hyenand_backward_create(int ndim, const int *dims, int B, int C, int mode, int dtype);
int hyenand_backward(hyenand_grad *grad, const void *q, const void *k, const void *v, const void *h,
                     long long h_batch_stride_elems, const void *dy, void *dq, void *dk, void *dv, void *dh,
                     void *cuda_stream);
long long hyenand_backward_guard_damage(hyenand_grad *grad);
void hyenand_backward_destroy(hyenand_grad *grad);

/*
 * Kernel synthesis: evaluates the input-dependent convolution kernel of Section 3.2.1 / 3.2.2,
 *
 *     K(x)[b][c][i] = w_c(c_i) * f_theta(c_i; gamma_b, beta_b)[c],
 *
 * on the tap grid and writes it as h in the layout hyenand_forward reads ([B][C][K_1]..[K_N], I/O dtype).
 * f_theta is the SIREN of Eq. 3 with `layers` hidden layers of width `hidden` and a frequency VECTOR omega0,
 * FiLM-modulated after every sine (Eq. 4):
 *     a_1 = gamma_1 * sin(omega0 * (W1 c_i + b1)) + beta_1,   a_j = gamma_j * sin(Wh_j a_{j-1} + bh_j) + beta_j,
 *     f = Wout a_J + bout.
 * Eq. 3 prints no biases: pass zeros for it.  gamma, beta ([B][layers][hidden]) are what the FiLM network makes of
 * the control variable z(x) (that small per-sample network is the caller's); NULL for both = identity modulation,
 * the static kernel.  w is the Gaussian window of Eq. 6 with window = sigma [N][C] (per axis and channel), or, for
 * mode CAUSAL, exp(-alpha_c |c_i|) with window = alpha [C] (Appendix A.3; taps exist only for displacements >= 0).
 * Coordinates per axis: LINEAR displacement d in [-(L-1), L-1] -> d/(L-1); CAUSAL t -> t/(L-1); CIRCULAR tap m ->
 * (m <= L/2 ? m : m - L) / (L/2); 0 when L = 1.  Window and SIREN share them.
 * All parameter arrays are fp32 DEVICE pointers, row-major: W1 [hidden][N], b1 [hidden], omega0 [hidden],
 * Wh [layers-1][hidden][hidden], bh [layers-1][hidden], Wout [C][hidden], bout [C].  hidden <= 64, layers <= 8.
 * fp32 arithmetic with accurate sine and exponential; the error of the first sine grows with |omega0 (W1 c + b1)|
 * (fp32 carries relative precision), about 1e-7 per radian.  Enqueues one kernel on cuda_stream; no allocation.
 */
int hyenand_synthesize_kernel(int ndim, const int *dims, int mode, int B, int C, int hidden, int layers,
                              const float *W1, const float *b1, const float *omega0, const float *Wh, const float *bh,
                              const float *Wout, const float *bout, const float *gamma, const float *beta,
                              const float *window, int dtype, void *h, void *cuda_stream);
/* The hidden and output layers of the network run on the tensor cores (tcgen05.mma, tf32 operands split in two so
 * that the products keep fp32 accuracy) wherever the operands fit in shared memory; the one wait of that kernel is
 * bounded.  Returns 0, or 1 once such a wait has given up since the library was loaded (the call that met it stored
 * an incomplete kernel), -1 if the word cannot be read.  Synchronises the device.  HYENAND_SYNTH_ALU in the
 * environment (read at the first call) selects the version without tensor cores. */
int hyenand_synth_device_status(void);


/*
 * Forward pass that allocates nothing (no counterpart in the paper: an integration aid).
 *
 * For callers that cannot allocate device memory when they need the operator -- host code running
 * while another thread captures a CUDA graph, code inside a memory pool's own critical section, a
 * service whose device memory was handed out completely at start-up.  There is no plan: the
 * geometry is passed with every call, and the workspace (twiddle table and half spectra, the same
 * passes as the general N-D path) lives in a fixed array of hyenand_noalloc_max_bytes() bytes
 * (16 MiB) inside the library image, which every GPU that loads the library holds until the
 * process exits.  Arguments and checks as hyenand_create_plan + hyenand_forward_ex (y must not overlap an
 * input); q, k, v, h, y are DEVICE pointers owned by the caller.  Work is enqueued on cuda_stream; the call
 * does not synchronise.
 *
 * Limits: every dims[n] <= 4096; one (b,c) slice's spectra (plus, when the filter is shared over
 * the batch, all C filter spectra) must fit the array, else HYENAND_ERR_UNSUPPORTED with the
 * sizes in hyenand_last_error().  Larger batches are processed in as many passes as needed.
 * The first call on a device resolves the array's device address (cudaGetSymbolAddress), and the
 * first call for a new geometry or dtype loads the kernels it needs and sets their attributes: make one
 * warm-up call per geometry and dtype before any stream capture.  All calls share the one array, which keeps
 * the previous call's contents (nothing in it needs to start at zero): calls that overlap on
 * the GPU (different streams, or different host threads) race and give wrong results; calls
 * on one stream are safe.  Neither cudaMalloc, cudaFree nor any allocating library routine is
 * called.
 */
size_t hyenand_noalloc_max_bytes(void);
int hyenand_forward_noalloc(int ndim, const int *dims, int B, int C, int causal, int dtype,
                            const void *q, const void *k, const void *v, const void *h,
                            long long h_batch_stride_elems, void *y, void *cuda_stream);

/*
 * Per-kernel accounting, for benchmarks.  Kernel ids run from 0 to
 * hyenand_plan_kernel_count()-1.  hyenand_plan_kernel_info gives, for one
 * forward of this plan (h_shared: filter shared over the batch or not), the
 * kernel's name, how often it is launched, and the ALGORITHMIC bytes and flops
 * of all its launches together: bytes = its inputs read once plus its outputs
 * written once; flops = 5 N log2 N per complex N-point line transform it
 * performs (un-pruned count) plus 12 per padded bin where it multiplies
 * spectra.  A kernel this plan never launches reports zeros.
 * hyenand_plan_set_timing(plan, 1) makes every later forward bracket each
 * kernel launch with CUDA events on the launching stream (and clears the
 * totals); with 2 instead of 1 the groups of a plan with several lanes are
 * additionally enqueued one after the other on the caller's stream, so that a
 * kernel's duration is its own and not stretched by another lane's kernels
 * sharing the GPU; 0 switches timing off. hyenand_plan_kernel_time returns the accumulated device time and
 * launch count of one kernel and must only be called after the stream has
 * been synchronised.  At most 4096 launches are recorded between two calls of
 * hyenand_plan_kernel_time.
 */
int hyenand_plan_kernel_count(const hyenand_plan *plan);
int hyenand_plan_kernel_info(const hyenand_plan *plan, int kernel_id, int h_shared, const char **name,
                             double *launches, double *bytes, double *flops);
int hyenand_plan_set_timing(hyenand_plan *plan, int enable);
int hyenand_plan_kernel_time(hyenand_plan *plan, int kernel_id, double *total_ms, double *launches);

#ifdef __cplusplus
}
#endif
#endif /* HYENAND_H */
