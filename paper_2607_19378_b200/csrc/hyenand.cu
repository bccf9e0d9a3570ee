// C ABI of the library: plan construction, argument checking, pass scheduling.
// See include/hyenand.h for the contract of every entry point.
#include <math.h>
#include <stdarg.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <vector>

#include "../../include/hyenand.h"
#include "common.cuh"
#include "ct1d.cuh"
#include "planes.cuh"
#include "core_tma.cuh"
#include "tma_util.cuh"
#include "fused2d.cuh"
#include "mixer.cuh"
#include "synth.cuh"
#include "backward.cuh"

using namespace hn;

static thread_local char g_err[512] = "";
static thread_local int g_code = 0;

static int fail(int code, const char *fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
    g_code = code;
    return code;
}

// Checked build: the address ranges a call may touch (the caller's tensors, the device allocations of the objects
// involved), handed to every translation unit before the call's kernels are enqueued.
struct DbgScope {
#ifdef HYENAND_DEBUG
    DbgRanges r;
    DbgScope() { r.n = 0; }
    void add(const void *ptr, size_t bytes)
    {
        if (ptr && bytes && r.n < kDbgRanges) { r.lo[r.n] = (unsigned long long)ptr; r.hi[r.n] = r.lo[r.n] + bytes; ++r.n; }
    }
    void add(const GuardedAllocs &g)
    {
        for (int i = 0; i < g.n; ++i) add(g.recs[i].base + kGuardBytes, g.recs[i].bytes);
    }
    void commit()
    {
        cudaDeviceSynchronize();               // kernels of earlier calls still compare against the previous list
        dbg_set_ranges(r);
    }
#else
    void add(const void *, size_t) {}
    void add(const GuardedAllocs &) {}
    void commit() {}
#endif
};

extern "C" int hyenand_debug_build(void)
{
#ifdef HYENAND_DEBUG
    return 1;
#else
    return 0;
#endif
}

extern "C" long long hyenand_debug_violations(unsigned long long *first_address, int *first_line, const char **file)
{
#ifdef HYENAND_DEBUG
    cudaDeviceSynchronize();
    const DbgReport rep = dbg_collect();
    if (first_address) *first_address = rep.first_address;
    if (first_line) *first_line = rep.first_line;
    if (file) *file = rep.file ? rep.file : "";
    return (long long)rep.count;
#else
    if (first_address) *first_address = 0;
    if (first_line) *first_line = 0;
    if (file) *file = "";
    return -1;
#endif
}

extern "C" long long hyenand_debug_selftest(void)
{
#ifdef HYENAND_DEBUG
    // Two valid buffers; only the first is registered.  Filling the first must count nothing, filling the second
    // must count every element: no access leaves allocated memory, so nothing faults.
    float *a = nullptr, *b = nullptr;
    const long long n = 1000;
    if (cudaMalloc(&a, n * sizeof(float)) != cudaSuccess) return -2;
    if (cudaMalloc(&b, n * sizeof(float)) != cudaSuccess) { cudaFree(a); return -2; }
    cudaDeviceSynchronize();
    (void)dbg_collect();
    DbgScope d;
    d.add(a, n * sizeof(float));
    d.commit();
    launch_fill(a, 1.f, n, nullptr);
    cudaDeviceSynchronize();
    const DbgReport clean = dbg_collect();
    launch_fill(b, 1.f, n, nullptr);
    cudaDeviceSynchronize();
    const DbgReport dirty = dbg_collect();
    cudaFree(a); cudaFree(b);
    if (clean.count != 0) return -3;
    if (dirty.first_address < (unsigned long long)b || dirty.first_address >= (unsigned long long)(b + n)) return -4;
    return (long long)dirty.count;
#else
    return -1;
#endif
}

enum Path { PATH_ND_GENERIC = 0, PATH_CT1D = 1, PATH_PLANES3D = 2, PATH_FUSED2D = 3 };
constexpr int kMaxLanes = 4;

struct hyenand_plan {
    int ndim, B, C, causal, dtype;
    bool circular;                    // periodic boundaries: K_n = P_n = L_n
    int dims[3];
    int L[3], K[3], P[3], log2p[3];   // internal 3-axis form (leading axes of extent 1)
    int XH;                           // half-spectrum bins along the contiguous axis
    int XP;                           // pitch of a half-spectrum row in the generic path (even)
    long long vol, kvol;              // elements per slice of q/k/v/y and of h
    int path;
    int device;
    // generic and plane paths: the batch is worked off in groups of slices_per_chunk slices; group i runs on
    // lane i % n_lanes.  A lane is a workspace set plus (when n_lanes > 1) a stream of the plan, so that the
    // short kernels of neighbouring groups overlap while each group's spectra stay close to the L2 cache.
    long long slices_per_chunk;
    long long ws_a_slice, ws_b_slice, wh_a_slice, wh_b_slice;   // float2 elements per slice
    int n_lanes;
    struct Lane {
        float2 *ws_a, *ws_b, *wh_a, *wh_b;
        long long wh_slices;          // slices the filter workspace holds (lane 0 also serves a filter shared over the batch)
        CoreTmaMaps tma;              // core maps: own k*v spectra, own filter spectra
        CoreTmaMaps tma_sh;           // own k*v spectra, lane 0's filter spectra (shared filter, lanes > 0)
        cudaStream_t st;              // nullptr: the caller's stream (n_lanes == 1)
        cudaEvent_t done;
    } lane[kMaxLanes];
    cudaEvent_t ev_fork;
    float2 *gtw;
    int gtw_n;
    int *dev_status;                  // device word set by a kernel whose bounded wait gave up
    Switches sw;
    GuardedAllocs allocs;
    bool serial_timing;               // per-kernel timing with the lanes run one after the other
    // slices [r0, r1) the next forward works on (the whole batch except inside hyenand_forward_host's pipeline)
    long long r0, r1;
    cudaStream_t copy_in, copy_out;   // streams of hyenand_forward_host's pipeline (created on first use)
    cudaEvent_t ev_in[2], ev_out;
    // long 1-D path
    Ct1dPlan ct;
    // host-staging for hyenand_forward_host
    void *stage[5];
    size_t stage_bytes[5];
    int h_dtype;                      // element type of the filter taps (differs from dtype only inside the mixer)
    // Element types per signal side on the multi-kernel paths, which take them per launch (the backward pass reads the
    // caller's bf16 tensors and writes a bf16 gradient on one side, an fp32 intermediate on the other): k and v are
    // `in`, the gate q and the result y are `out`.  Equal to dtype everywhere else.
    int dt_in, dt_out, dt_in2, dt_out2;
    // Second signal side of the multi-kernel paths (backward pass): after y = q (h conv (k v)) every group also
    // computes y2 = q2 (h' conv (k2 v2)) with h'[d] = h[-d], whose spectrum is the conjugate of the filter spectrum
    // the group has just computed.  Unused (nullptr) in an ordinary forward.
    const char *q2, *k2, *v2;
    char *y2;
    const char *qg2;                  // a second gate and result of the same convolution, yg2 = qg2 * (h conv (k v)): of the one
    char *yg2;                        // forward on the fused 2-D path, of the second signal side on the multi-kernel paths
    size_t ws_bytes;
    Prof prof;
};

static int next_pow2_log(int x)
{
    int l = 0;
    while ((1 << l) < x) ++l;
    return l;
}

static size_t elsize(int dtype) { return dtype == HYENAND_F32 ? 4 : 2; }

static int dev_alloc(hyenand_plan *p, void **ptr, size_t bytes)
{
    if (bytes == 0) bytes = 16;
    cudaError_t e = guarded_alloc(&p->allocs, ptr, bytes);
    if (e != cudaSuccess) {
        cudaGetLastError();
        *ptr = nullptr;
        return fail(HYENAND_ERR_ALLOC, "cudaMalloc of %zu bytes failed: %s", bytes, cudaGetErrorString(e));
    }
    p->ws_bytes += bytes;
    return HYENAND_OK;
}

extern "C" const char *hyenand_last_error(void) { return g_err; }
extern "C" int hyenand_last_error_code(void) { return g_err[0] ? g_code : HYENAND_OK; }

extern "C" void hyenand_destroy_plan(hyenand_plan *p)
{
    if (!p) return;
    int cur = 0;
    cudaGetDevice(&cur);
    if (cur != p->device) cudaSetDevice(p->device);
    guarded_free_all(&p->allocs);            // workspace sets, twiddle tables, status word (cudaFree synchronises)
    for (int l = 0; l < kMaxLanes; ++l) {
        if (p->lane[l].st) cudaStreamDestroy(p->lane[l].st);
        if (p->lane[l].done) cudaEventDestroy(p->lane[l].done);
    }
    if (p->ev_fork) cudaEventDestroy(p->ev_fork);
    for (int i = 0; i < 5; ++i) cudaFree(p->stage[i]);
    if (p->copy_in) cudaStreamDestroy(p->copy_in);
    if (p->copy_out) cudaStreamDestroy(p->copy_out);
    for (int i = 0; i < 2; ++i) if (p->ev_in[i]) cudaEventDestroy(p->ev_in[i]);
    if (p->ev_out) cudaEventDestroy(p->ev_out);
    p->prof.destroy();
    if (cur != p->device) cudaSetDevice(cur);
    delete p;
}

static AxisArgs planes3d_core_args(const hyenand_plan *p, int lane, long long n, bool shared, long long s0, bool conj = false);
static void make_core_maps(hyenand_plan *p);
static AxisArgs generic_core_args(const hyenand_plan *p, int lane, long long n, bool shared, long long s0, bool conj = false);
static void choose_groups(hyenand_plan *p, long long per_slice_elems);

extern "C" hyenand_plan *hyenand_create_plan(int ndim, const int *dims, int B, int C, int causal, int dtype)
{
    if (causal != 0 && causal != 1) { g_err[0] = 0; fail(HYENAND_ERR_INVALID_ARG, "causal must be 0 or 1"); return nullptr; }
    return hyenand_create_plan_mode(ndim, dims, B, C, causal ? HYENAND_MODE_CAUSAL : HYENAND_MODE_LINEAR, dtype);
}

extern "C" hyenand_plan *hyenand_create_plan_mode(int ndim, const int *dims, int B, int C, int mode, int dtype)
{
    g_err[0] = 0;
    if (mode != HYENAND_MODE_LINEAR && mode != HYENAND_MODE_CAUSAL && mode != HYENAND_MODE_CIRCULAR) {
        fail(HYENAND_ERR_INVALID_ARG, "unknown boundary mode %d", mode);
        return nullptr;
    }
    const int causal = mode == HYENAND_MODE_CAUSAL;
    const bool circular = mode == HYENAND_MODE_CIRCULAR;
    if (ndim < 1 || ndim > 3) { fail(HYENAND_ERR_INVALID_ARG, "ndim must be 1, 2 or 3 (got %d)", ndim); return nullptr; }
    if (!dims) { fail(HYENAND_ERR_INVALID_ARG, "dims is NULL"); return nullptr; }
    if (B < 1 || C < 1) { fail(HYENAND_ERR_INVALID_ARG, "B and C must be >= 1 (got %d, %d)", B, C); return nullptr; }
    if (dtype != HYENAND_F32 && dtype != HYENAND_BF16) { fail(HYENAND_ERR_INVALID_ARG, "unknown dtype %d", dtype); return nullptr; }
    for (int a = 0; a < ndim; ++a)
        if (dims[a] < 1) { fail(HYENAND_ERR_INVALID_ARG, "dims[%d] = %d must be >= 1", a, dims[a]); return nullptr; }
    if (causal && ndim != 1) { fail(HYENAND_ERR_UNSUPPORTED, "causal kernels are defined for 1-D grids only"); return nullptr; }
    if (circular)
        for (int a = 0; a < ndim; ++a)
            if (dims[a] & (dims[a] - 1)) {
                fail(HYENAND_ERR_UNSUPPORTED, "circular mode transforms the grid itself: dims[%d] = %d is not a power of two", a, dims[a]);
                return nullptr;
            }

    hyenand_plan *p = new hyenand_plan();
    memset(p, 0, sizeof(*p));
    p->ndim = ndim; p->B = B; p->C = C; p->causal = causal; p->circular = circular; p->dtype = dtype; p->h_dtype = dtype;
    p->dt_in = p->dt_out = p->dt_in2 = p->dt_out2 = dtype;
    p->r0 = 0; p->r1 = (long long)B * C;
    cudaGetDevice(&p->device);
    p->sw = read_switches();
    p->prof.nvtx = p->sw.nvtx;
    p->n_lanes = 1;
    p->vol = 1; p->kvol = 1;
    for (int a = 0; a < 3; ++a) { p->L[a] = 1; p->K[a] = 1; p->P[a] = 1; p->log2p[a] = 0; }
    for (int a = 0; a < ndim; ++a) {
        const int ia = 3 - ndim + a;
        p->dims[a] = dims[a];
        if ((long long)dims[a] > (1ll << 25)) { fail(HYENAND_ERR_UNSUPPORTED, "dims[%d] too long", a); delete p; return nullptr; }
        p->L[ia] = dims[a];
        p->K[ia] = (causal || circular) ? dims[a] : 2 * dims[a] - 1;
        p->log2p[ia] = circular ? next_pow2_log(dims[a]) : next_pow2_log(2 * dims[a] - 1);
        p->P[ia] = 1 << p->log2p[ia];
        p->vol *= dims[a];
        p->kvol *= p->K[ia];
    }
    p->XH = p->P[2] / 2 + 1;
    p->XP = (p->XH + 1) & ~1;
    if (circular) {
        // periodic boundaries run on the general N-D passes, which transform whole lines here (nothing is
        // padded, so there is no zero half to prune and no half to crop); no plane, fused or tensor-copy kernels
        p->sw.force_generic = p->sw.no_tma = true;
    }

    if (ndim == 1 && p->log2p[2] > kMaxLineLog2 && !circular) {
        p->path = PATH_CT1D;
        if (p->log2p[2] > 24) { fail(HYENAND_ERR_UNSUPPORTED, "1-D grid too long (padded size 2^%d > 2^24)", p->log2p[2]); delete p; return nullptr; }
        size_t bytes = 0;
        int e = ct1d_init(&p->ct, p->L[2], p->K[2], p->log2p[2], B, C, causal, dtype, p->sw, &p->allocs, &bytes);
        if (e != HYENAND_OK) {
            fail(e, "long 1-D path: workspace allocation failed (%zu bytes were allocated before): %s", bytes,
                 cudaGetErrorString(cudaGetLastError()));
            hyenand_destroy_plan(p); return nullptr;
        }
        p->ws_bytes += bytes;
        if (dev_alloc(p, (void **)&p->dev_status, sizeof(int)) || cudaMemset(p->dev_status, 0, sizeof(int)) != cudaSuccess) {
            hyenand_destroy_plan(p);
            return nullptr;
        }
        p->ct.status = p->dev_status;
        return p;
    }
    for (int a = 0; a < 3; ++a)
        if (p->log2p[a] > kMaxLineLog2) {
            fail(HYENAND_ERR_UNSUPPORTED, "padded axis of %d points exceeds the limit of %d for ndim >= 2",
                 p->P[a], 1 << kMaxLineLog2);
            delete p; return nullptr;
        }

    p->path = PATH_ND_GENERIC;
    const bool three = p->P[0] > 1;
    if (three && p->log2p[1] == p->log2p[2] && plane_supported(p->log2p[2]) && !p->sw.force_generic)
        p->path = PATH_PLANES3D;
    if (ndim == 2 && p->log2p[1] == p->log2p[2] && fused2d_supported(p->log2p[2]) && !p->sw.force_generic)
        p->path = PATH_FUSED2D;
    if (p->path == PATH_FUSED2D) {
        p->ws_a_slice = p->wh_a_slice = p->ws_b_slice = p->wh_b_slice = 0;   // nothing leaves the chip
    } else if (p->path == PATH_PLANES3D) {
        // spectra [plane][XH][P_y]; the z pass works in place on the k*v spectra
        p->ws_a_slice = (long long)p->L[0] * p->XH * p->P[1];
        p->wh_a_slice = (long long)p->K[0] * p->XH * p->P[1];
        p->ws_b_slice = p->wh_b_slice = 0;
    } else {
        p->ws_a_slice = (long long)p->L[0] * p->L[1] * p->XP;
        p->wh_a_slice = (long long)p->K[0] * p->K[1] * p->XP;
        p->ws_b_slice = three ? (long long)p->L[0] * p->P[1] * p->XP : 0;
        p->wh_b_slice = three ? (long long)p->K[0] * p->P[1] * p->XP : 0;
    }
    const long long per_slice = p->ws_a_slice + p->ws_b_slice + p->wh_a_slice + p->wh_b_slice;
    choose_groups(p, per_slice);
    const long long spc = p->slices_per_chunk;

    int gl = 1;
    for (int a = 0; a < 3; ++a) if (p->log2p[a] > gl) gl = p->log2p[a];
    p->gtw_n = 1 << gl;
    std::vector<float2> tw(p->gtw_n);
    for (int t = 0; t < p->gtw_n; ++t) {
        const double ang = -2.0 * M_PI * (double)t / (double)p->gtw_n;
        tw[t] = make_float2((float)cos(ang), (float)sin(ang));
    }
    int e = dev_alloc(p, (void **)&p->gtw, sizeof(float2) * p->gtw_n);
    for (int l = 0; l < p->n_lanes && !e; ++l) {
        hyenand_plan::Lane &ln = p->lane[l];
        ln.wh_slices = spc;                                 // (a filter shared over the batch gets room for all channels on first use)
        e = dev_alloc(p, (void **)&ln.ws_a, sizeof(float2) * p->ws_a_slice * spc);
        if (!e && p->ws_b_slice) e = dev_alloc(p, (void **)&ln.ws_b, sizeof(float2) * p->ws_b_slice * spc);
        if (!e) e = dev_alloc(p, (void **)&ln.wh_a, sizeof(float2) * p->wh_a_slice * ln.wh_slices);
        if (!e && p->wh_b_slice) e = dev_alloc(p, (void **)&ln.wh_b, sizeof(float2) * p->wh_b_slice * ln.wh_slices);
    }
    if (!e && cudaMemcpy(p->gtw, tw.data(), sizeof(float2) * p->gtw_n, cudaMemcpyHostToDevice) != cudaSuccess)
        e = fail(HYENAND_ERR_CUDA, "twiddle upload failed: %s", cudaGetErrorString(cudaGetLastError()));
    if (!e) e = dev_alloc(p, (void **)&p->dev_status, sizeof(int));
    if (!e && cudaMemset(p->dev_status, 0, sizeof(int)) != cudaSuccess)
        e = fail(HYENAND_ERR_CUDA, "status word: %s", cudaGetErrorString(cudaGetLastError()));
    if (!e && p->n_lanes > 1) {
        bool ok = cudaEventCreateWithFlags(&p->ev_fork, cudaEventDisableTiming) == cudaSuccess;
        for (int l = 0; l < p->n_lanes && ok; ++l)
            ok = cudaStreamCreateWithFlags(&p->lane[l].st, cudaStreamNonBlocking) == cudaSuccess &&
                 cudaEventCreateWithFlags(&p->lane[l].done, cudaEventDisableTiming) == cudaSuccess;
        if (!ok) e = fail(HYENAND_ERR_CUDA, "lane streams: %s", cudaGetErrorString(cudaGetLastError()));
    }
    if (e) { hyenand_destroy_plan(p); return nullptr; }
    make_core_maps(p);
    return p;
}

// tensor maps of the fused core's buffers; left invalid where the TMA core does not apply
static void make_core_maps(hyenand_plan *p)
{
    if (p->path != PATH_PLANES3D && p->path != PATH_ND_GENERIC) return;
    if (p->sw.no_tma) return;
    const long long spc = p->slices_per_chunk;
    for (int l = 0; l < p->n_lanes; ++l) {
        hyenand_plan::Lane &ln = p->lane[l];
        const AxisArgs own = p->path == PATH_PLANES3D ? planes3d_core_args(p, l, spc, false, 0)
                                                      : generic_core_args(p, l, spc, false, 0);
        core_tma_make(&ln.tma, own, spc, ln.wh_slices);
        if (l > 0) {
            const AxisArgs sh = p->path == PATH_PLANES3D ? planes3d_core_args(p, l, spc, true, 0)
                                                         : generic_core_args(p, l, spc, true, 0);
            core_tma_make(&ln.tma_sh, sh, spc, p->lane[0].wh_slices);
        }
    }
}

// The multi-kernel paths (long 1-D included) transform the filter in kernels of their own, which take the taps' element type per launch:
// a plan of fp32 tensors can read bf16 taps there (the mixer's inner plan: q, k, v come out of its fp32 pointwise
// stage, the kernel arrives in the caller's type).  False where the path has one element type for everything.
static bool plan_set_filter_dtype(hyenand_plan *p, int dtype)
{
    if (dtype == p->dtype) { p->h_dtype = dtype; return true; }
    if (p->path == PATH_CT1D) {
        if (!ct1d_takes_dtype(&p->ct, dtype)) return false;
    } else if (p->path != PATH_PLANES3D && p->path != PATH_ND_GENERIC) {
        return false;
    }
    p->h_dtype = dtype;
    return true;
}

// A filter shared over the batch is transformed once per forward, all C channels into lane 0's filter workspace,
// which therefore needs room for C slices instead of one group's: it is enlarged the first time such a forward is
// asked for (plans used with per-sample filters never pay for it).
static int ensure_shared_filter_room(hyenand_plan *p)
{
    hyenand_plan::Lane &ln = p->lane[0];
    if (ln.wh_slices >= p->C) return 0;
    float2 *a = nullptr, *b = nullptr;
    int e = dev_alloc(p, (void **)&a, sizeof(float2) * p->wh_a_slice * p->C);
    if (!e && p->wh_b_slice) e = dev_alloc(p, (void **)&b, sizeof(float2) * p->wh_b_slice * p->C);
    if (e) return e;
    ln.wh_a = a; ln.wh_b = b; ln.wh_slices = p->C;       // (the smaller buffers stay with the plan until it is destroyed)
#ifdef HYENAND_DEBUG
    cudaDeviceSynchronize();
    dbg_append_range(a, sizeof(float2) * p->wh_a_slice * p->C);
    if (b) dbg_append_range(b, sizeof(float2) * p->wh_b_slice * p->C);
#endif
    make_core_maps(p);
    return 0;
}

// Group size and number of lanes.  HYENAND_GROUP_SLICES / HYENAND_LANES override the choice (development aids,
// read at plan creation like the other switches).
static void choose_groups(hyenand_plan *p, long long per_slice_elems)
{
    const long long S = (long long)p->B * p->C;
    long long spc = S;
    int lanes = 1;
    if (per_slice_elems > 0) {
        // A lane's workspace stays under 1 GiB.  A batch that needs several groups runs them on two lanes, in
        // groups of equal size: measured on B200 this is as fast as one launch over the whole batch or slightly
        // faster (volume3d 5.38 vs 5.48 ms, pde2d 2.70 vs 2.78 ms) at a fraction of the workspace, while groups
        // small enough to keep their spectra in the L2 cache are slower (launches that do not fill the GPU).
        const long long slice_bytes = per_slice_elems * (long long)sizeof(float2);
        long long most = (1ll << 30) / slice_bytes;
        if (most < 1) most = 1;
        if (most < S) {
            lanes = 2;
            long long groups = (S + most - 1) / most;
            groups = (groups + lanes - 1) / lanes * lanes;
            spc = (S + groups - 1) / groups;
        }
    }
    if (const char *e = getenv("HYENAND_GROUP_SLICES")) { const long long v = atoll(e); if (v > 0) spc = v; }
    if (const char *e = getenv("HYENAND_LANES")) { const int v = atoi(e); if (v >= 1 && v <= kMaxLanes) lanes = v; }
    if (spc < 1) spc = 1;
    if (spc > S) spc = S;
    if ((S + spc - 1) / spc < lanes) lanes = (int)((S + spc - 1) / spc);
    if (per_slice_elems == 0) lanes = 1;
    p->slices_per_chunk = spc;
    p->n_lanes = lanes;
}

extern "C" int hyenand_plan_device_status(hyenand_plan *p)
{
    g_err[0] = 0;
    if (!p) { fail(HYENAND_ERR_INVALID_ARG, "plan is NULL"); return -1; }
    if (!p->dev_status) return 0;             // plans whose kernels make no such waits have no status word
    int v = 0;
    if (cudaMemcpy(&v, p->dev_status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) {
        fail(HYENAND_ERR_CUDA, "reading the status word failed: %s", cudaGetErrorString(cudaGetLastError()));
        return -1;
    }
    return v;
}

extern "C" long long hyenand_plan_guard_damage(hyenand_plan *p)
{
    g_err[0] = 0;
    if (!p) { fail(HYENAND_ERR_INVALID_ARG, "plan is NULL"); return -1; }
    const long long bad = guard_damage(&p->allocs);
    if (bad < 0) fail(HYENAND_ERR_CUDA, "reading the guard bands failed: %s", cudaGetErrorString(cudaGetLastError()));
    return bad;
}

extern "C" int hyenand_selftest_bounded_wait(int polls)
{
    g_err[0] = 0;
    const int v = tma_selftest_bounded_wait(polls);
    if (v < 0) fail(HYENAND_ERR_CUDA, "bounded-wait self-test could not run: %s", cudaGetErrorString(cudaGetLastError()));
    return v;
}

// ---- scheduling of the multi-kernel paths -------------------------------------------------------

// Lanes: group i of the batch runs on lane i % n_lanes.  With one lane everything is enqueued on the caller's
// stream.  With several, the lanes' own streams start after the work already queued on the caller's stream
// (fork event) and the caller's stream continues after all of them (join events): to the caller the forward
// still looks like work enqueued on its stream.
// (While per-kernel timing in its serialised mode is on, every lane uses the caller's stream, so that kernel
// durations are not stretched by kernels of the other lanes sharing the GPU.)
static bool lanes_concurrent(const hyenand_plan *p) { return p->n_lanes > 1 && !(p->prof.on && p->serial_timing); }
static cudaStream_t lane_stream(hyenand_plan *p, int l, cudaStream_t st) { return lanes_concurrent(p) ? p->lane[l].st : st; }

static int lanes_fork(hyenand_plan *p, cudaStream_t st)
{
    if (!lanes_concurrent(p)) return 0;
    if (cudaEventRecord(p->ev_fork, st) != cudaSuccess) return -1;
    for (int l = 0; l < p->n_lanes; ++l)
        if (cudaStreamWaitEvent(p->lane[l].st, p->ev_fork, 0) != cudaSuccess) return -1;
    return 0;
}

static int lanes_join(hyenand_plan *p, cudaStream_t st)
{
    if (!lanes_concurrent(p)) return 0;
    for (int l = 0; l < p->n_lanes; ++l)
        if (cudaEventRecord(p->lane[l].done, p->lane[l].st) != cudaSuccess ||
            cudaStreamWaitEvent(st, p->lane[l].done, 0) != cudaSuccess)
            return -1;
    return 0;
}

// one transform along the middle axis: warp-engine kernel where it applies, else the block-wide one
static int launch_axis_any(const Switches &sw, const AxisArgs &a, int mode, cudaStream_t st)
{
    if (core_w_supported(a.log2p) && !sw.generic_core) {
        const int c = launch_axis_w(a, mode == AXIS_INV, st);
        if (c >= 0) return c;
    }
    return launch_axis(a, mode, st);
}

static int filter_spectrum_generic(hyenand_plan *p, int l, const char *h, long long n_slices, cudaStream_t st, int *launches)
{
    hyenand_plan::Lane &ln = p->lane[l];
    // rows of h, then (3-D) the middle axis
    RowsArgs r{};
    r.a = h; r.b = nullptr; r.out = ln.wh_a; r.pitch = p->XP;
    r.rows = n_slices * p->K[0] * p->K[1];
    r.len = p->K[2];
    r.shift = (p->causal || p->circular) ? 0 : p->L[2] - 1;
    r.log2p = p->log2p[2];
    r.prune_in = p->causal && p->P[2] >= 2;
    r.full_in = p->circular;
    r.gtw = p->gtw; r.gtw_n = p->gtw_n;
    p->prof.begin(KID_ROWS_H, st);
    const bool roww = rows_w_supported(r.log2p) && !p->sw.generic_rows;
    int n = roww ? launch_rows_fwd_w(r, p->h_dtype, st) : launch_rows_fwd(r, p->h_dtype, st);
    p->prof.end(st);
    if (n < 0) return -1;
    *launches += n;
    if (p->P[0] > 1) {
        AxisArgs a{};
        a.in = ln.wh_a; a.out = ln.wh_b;
        a.n_outer = n_slices * p->K[0];
        a.in_outer = (long long)p->K[1] * p->XP;
        a.out_outer = (long long)p->P[1] * p->XP;
        a.nc = p->XP; a.n_in = p->K[1]; a.n_out = p->P[1];
        a.shift = p->circular ? 0 : p->L[1] - 1; a.log2p = p->log2p[1]; a.prune_in = 0;
        a.gtw = p->gtw; a.gtw_n = p->gtw_n;
        p->prof.begin(KID_AXIS_H, st);
        n = launch_axis_any(p->sw, a, AXIS_FWD, st);
        p->prof.end(st);
        if (n < 0) return -1;
        *launches += n;
    }
    return 0;
}

// arguments of the fused core (last transformed axis) of the generic path for n slices starting at slice s0,
// in the workspace of lane l (a filter shared over the batch sits in lane 0's filter workspace)
static AxisArgs generic_core_args(const hyenand_plan *p, int l, long long n, bool shared, long long s0, bool conj)
{
    const hyenand_plan::Lane &ln = p->lane[l], &lh = p->lane[shared ? 0 : l];
    const bool three = p->P[0] > 1;
    AxisArgs a{};
    const int ax = three ? 0 : 1;                       // core axis
    const long long inner = three ? (long long)p->P[1] * p->XP : p->XP;
    a.in = three ? ln.ws_b : ln.ws_a; a.out = (float2 *)a.in;
    a.n_outer = n;
    a.in_outer = a.out_outer = (long long)p->L[ax] * inner;
    a.nc = (int)inner; a.n_in = p->L[ax]; a.n_out = p->L[ax]; a.shift = 0;
    a.log2p = p->log2p[ax]; a.prune_in = 1; a.full = p->circular;
    a.h = three ? lh.wh_b : lh.wh_a;
    a.h_outer = (long long)p->K[ax] * inner;
    a.h_n_in = p->K[ax];
    a.h_shift = (p->causal || p->circular) ? 0 : p->L[ax] - 1;
    a.h_mod = shared ? p->C : 0;
    a.h_off = shared ? s0 % p->C : 0;
    a.scale = (float)(1.0 / ((double)p->P[0] * p->P[1] * p->P[2]));
    a.gtw = p->gtw; a.gtw_n = p->gtw_n;
    a.h_conj = conj;
    return a;
}

// the fused core of either multi-kernel path: tensor-copy version where the lane's maps apply, else the
// cp.async version, else the block-wide kernel
static int launch_core_any(hyenand_plan *p, int l, const AxisArgs &a, bool shared, cudaStream_t st)
{
    const hyenand_plan::Lane &ln = p->lane[l];
    const CoreTmaMaps &m = (shared && l > 0) ? ln.tma_sh : ln.tma;
    int c = -1;
    if (m.valid && !p->sw.no_tma) c = launch_core_tma(a, m, p->dev_status, st);
    if (c < 0)
        c = (core_w_supported(a.log2p) && !p->sw.generic_core) ? launch_core_w(a, st) : launch_axis(a, AXIS_CORE, st);
    return c;
}

static int forward_generic(hyenand_plan *p, const char *q, const char *k, const char *v, const char *h,
                           bool shared, char *y, cudaStream_t st0, int *launches)
{
    const size_t es = elsize(p->dtype);
    const bool three = p->P[0] > 1;
    if (shared && ensure_shared_filter_room(p)) return -2;
    if (shared && p->r0 == 0 && filter_spectrum_generic(p, 0, h, p->C, st0, launches)) return -1;
    if (lanes_fork(p, st0)) return -1;
    int g = 0;
    for (long long s0 = p->r0; s0 < p->r1; s0 += p->slices_per_chunk, ++g) {
        const int l = g % p->n_lanes;
        hyenand_plan::Lane &ln = p->lane[l];
        cudaStream_t st = lane_stream(p, l, st0);
        const long long n = p->r1 - s0 < p->slices_per_chunk ? p->r1 - s0 : p->slices_per_chunk;
        if (!shared && filter_spectrum_generic(p, l, h + (size_t)s0 * p->kvol * elsize(p->h_dtype), n, st, launches)) return -1;
        // one signal side: rows, [middle axis], core against the group's filter spectrum (or its conjugate), back
        auto side = [&](const char *sq, const char *sk, const char *sv, char *sy, bool conj, int dt_in, int dt_out,
                        const char *sq2, char *sy2) -> int {
            const size_t ei = elsize(dt_in), eo = elsize(dt_out);
            RowsArgs r{};
            r.a = sk + (size_t)s0 * p->vol * ei; r.b = sv + (size_t)s0 * p->vol * ei; r.out = ln.ws_a; r.pitch = p->XP;
            r.rows = n * p->L[0] * p->L[1]; r.len = p->L[2]; r.shift = 0; r.log2p = p->log2p[2];
            r.prune_in = 1; r.full_in = p->circular; r.gtw = p->gtw; r.gtw_n = p->gtw_n;
            p->prof.begin(KID_ROWS_U, st);
            const bool roww = rows_w_supported(r.log2p) && !p->sw.generic_rows;
            int c = roww ? launch_rows_fwd_w(r, dt_in, st) : launch_rows_fwd(r, dt_in, st);
            p->prof.end(st);
            if (c < 0) return -1;
            *launches += c;
            if (three) {
                AxisArgs a{};
                a.in = ln.ws_a; a.out = ln.ws_b;
                a.n_outer = n * p->L[0];
                a.in_outer = (long long)p->L[1] * p->XP; a.out_outer = (long long)p->P[1] * p->XP;
                a.nc = p->XP; a.n_in = p->L[1]; a.n_out = p->P[1]; a.shift = 0;
                a.log2p = p->log2p[1]; a.prune_in = p->P[1] >= 2 && !p->circular;
                a.gtw = p->gtw; a.gtw_n = p->gtw_n;
                p->prof.begin(KID_AXIS_U, st);
                c = launch_axis_any(p->sw, a, AXIS_FWD, st);
                p->prof.end(st);
                if (c < 0) return -1;
                *launches += c;
            }
            {
                const AxisArgs a = generic_core_args(p, l, n, shared, s0, conj);
                p->prof.begin(KID_CORE, st);
                c = launch_core_any(p, l, a, shared, st);
                p->prof.end(st);
                if (c < 0) return -1;
                *launches += c;
            }
            if (three) {
                AxisArgs a{};
                a.in = ln.ws_b; a.out = ln.ws_a;
                a.n_outer = n * p->L[0];
                a.in_outer = (long long)p->P[1] * p->XP; a.out_outer = (long long)p->L[1] * p->XP;
                a.nc = p->XP; a.n_in = p->P[1]; a.n_out = p->L[1]; a.shift = 0;
                a.log2p = p->log2p[1]; a.prune_in = 0; a.full = p->circular;
                a.gtw = p->gtw; a.gtw_n = p->gtw_n;
                p->prof.begin(KID_AXIS_INV, st);
                c = launch_axis_any(p->sw, a, AXIS_INV, st);
                p->prof.end(st);
                if (c < 0) return -1;
                *launches += c;
            }
            RowsInvArgs ri{};
            ri.in = ln.ws_a; ri.pitch = p->XP; ri.q = sq ? sq + (size_t)s0 * p->vol * eo : nullptr; ri.y = sy + (size_t)s0 * p->vol * eo;
            if (sy2) { ri.q2 = sq2 + (size_t)s0 * p->vol * eo; ri.y2 = sy2 + (size_t)s0 * p->vol * eo; }
            ri.rows = n * p->L[0] * p->L[1]; ri.len = p->L[2]; ri.log2p = p->log2p[2];
            ri.gtw = p->gtw; ri.gtw_n = p->gtw_n; ri.full_out = p->circular;
            p->prof.begin(KID_ROWS_INV, st);
            c = roww ? launch_rows_inv_w(ri, dt_out, st) : launch_rows_inv(ri, dt_out, st);
            p->prof.end(st);
            if (c < 0) return -1;
            *launches += c;
            return 0;
        };
        if (side(q, k, v, y, false, p->dt_in, p->dt_out, nullptr, nullptr)) return -1;
        if (p->y2 && side(p->q2, p->k2, p->v2, p->y2, true, p->dt_in2, p->dt_out2, p->qg2, p->yg2)) return -1;
    }
    return lanes_join(p, st0);
}

// arguments of the z core of the 3-D path for n slices starting at slice s0, in the workspace of lane l
static AxisArgs planes3d_core_args(const hyenand_plan *p, int l, long long n, bool shared, long long s0, bool conj)
{
    const hyenand_plan::Lane &ln = p->lane[l], &lh = p->lane[shared ? 0 : l];
    const long long nc = (long long)p->XH * p->P[1];
    AxisArgs a{};
    a.in = ln.ws_a; a.out = ln.ws_a;
    a.n_outer = n; a.in_outer = a.out_outer = (long long)p->L[0] * nc;
    a.nc = (int)nc; a.n_in = p->L[0]; a.n_out = p->L[0]; a.shift = 0;
    a.log2p = p->log2p[0]; a.prune_in = 1;
    a.h = lh.wh_a; a.h_outer = (long long)p->K[0] * nc; a.h_n_in = p->K[0]; a.h_shift = p->L[0] - 1;
    a.h_mod = shared ? p->C : 0; a.h_off = shared ? s0 % p->C : 0;
    // 1/P of the inverse transforms, and the factors 1/2 the two forward plane kernels leave out of their row separations
    a.scale = (float)(0.25 / ((double)p->P[0] * p->P[1] * p->P[2]));
    a.gtw = p->gtw; a.gtw_n = p->gtw_n;
    a.h_conj = conj;
    return a;
}

static int forward_planes3d(hyenand_plan *p, const char *q, const char *k, const char *v, const char *h,
                            bool shared, char *y, cudaStream_t st0, int *launches)
{
    const size_t es = elsize(p->dtype);
    auto filter = [&](int l, const char *hp, long long n, cudaStream_t st) -> int {
        PlaneArgs a{};
        a.a = hp; a.out = p->lane[l].wh_a; a.planes = n * p->K[0];
        a.a_elems = n * p->kvol;
        a.lx = p->L[2]; a.ly = p->L[1]; a.gtw = p->gtw; a.gtw_n = p->gtw_n;
        p->prof.begin(KID_PLANE_H, st);
        int c = launch_plane(a, PLANE_H, p->log2p[2], p->h_dtype, st);
        p->prof.end(st);
        if (c < 0) return -1;
        *launches += c;
        return 0;
    };
    if (shared && ensure_shared_filter_room(p)) return -2;
    if (shared && p->r0 == 0 && filter(0, h, p->C, st0)) return -1;
    if (lanes_fork(p, st0)) return -1;
    int g = 0;
    for (long long s0 = p->r0; s0 < p->r1; s0 += p->slices_per_chunk, ++g) {
        const int l = g % p->n_lanes;
        hyenand_plan::Lane &ln = p->lane[l];
        cudaStream_t st = lane_stream(p, l, st0);
        const long long n = p->r1 - s0 < p->slices_per_chunk ? p->r1 - s0 : p->slices_per_chunk;
        if (!shared && filter(l, h + (size_t)s0 * p->kvol * elsize(p->h_dtype), n, st)) return -1;
        // one signal side: k v planes, z core against the group's filter spectrum (or its conjugate), planes back
        auto side = [&](const char *sq, const char *sk, const char *sv, char *sy, bool conj, int dt_in, int dt_out,
                        const char *sq2, char *sy2) -> int {
            const size_t ei = elsize(dt_in), eo = elsize(dt_out);
            PlaneArgs u{};
            u.a = sk + (size_t)s0 * p->vol * ei; u.b = sv + (size_t)s0 * p->vol * ei; u.out = ln.ws_a;
            u.a_elems = n * p->vol;
            u.planes = n * p->L[0]; u.lx = p->L[2]; u.ly = p->L[1]; u.gtw = p->gtw; u.gtw_n = p->gtw_n;
            p->prof.begin(KID_PLANE_U, st);
            int c = launch_plane(u, PLANE_U, p->log2p[2], dt_in, st);
            p->prof.end(st);
            if (c < 0) return -1;
            *launches += c;
            const AxisArgs a = planes3d_core_args(p, l, n, shared, s0, conj);
            p->prof.begin(KID_CORE, st);
            c = launch_core_any(p, l, a, shared, st);
            p->prof.end(st);
            if (c < 0) return -1;
            *launches += c;
            PlaneArgs iv{};
            iv.a = sq ? sq + (size_t)s0 * p->vol * eo : nullptr; iv.y = sy + (size_t)s0 * p->vol * eo; iv.in = ln.ws_a;     // no gate: y = the convolution
            if (sy2) { iv.q2 = sq2 + (size_t)s0 * p->vol * eo; iv.y2 = sy2 + (size_t)s0 * p->vol * eo; }
            iv.planes = n * p->L[0]; iv.lx = p->L[2]; iv.ly = p->L[1]; iv.gtw = p->gtw; iv.gtw_n = p->gtw_n;
            p->prof.begin(KID_PLANE_INV, st);
            c = launch_plane(iv, PLANE_INV, p->log2p[2], dt_out, st);
            p->prof.end(st);
            if (c < 0) return -1;
            *launches += c;
            return 0;
        };
        if (side(q, k, v, y, false, p->dt_in, p->dt_out, nullptr, nullptr)) return -1;
        if (p->y2 && side(p->q2, p->k2, p->v2, p->y2, true, p->dt_in2, p->dt_out2, p->qg2, p->yg2)) return -1;
    }
    return lanes_join(p, st0);
}

static int forward_fused2d(hyenand_plan *p, const void *q, const void *k, const void *v, const void *h,
                           bool shared, void *y, cudaStream_t st, int *launches)
{
    Fused2dArgs a{};
    const size_t es = elsize(p->dtype);
    const size_t off = (size_t)p->r0 * p->vol * es;
    a.q = (const char *)q + off; a.k = (const char *)k + off; a.v = (const char *)v + off; a.y = (char *)y + off;
    a.h = shared ? h : (const void *)((const char *)h + (size_t)p->r0 * p->kvol * es);
    a.slices = p->r1 - p->r0; a.lx = p->L[2]; a.ly = p->L[1];
    a.h_mod = shared ? p->C : 0; a.h_off = shared ? p->r0 % p->C : 0;
    a.scale = (float)(1.0 / ((double)p->P[1] * p->P[2]));
    if (p->yg2) { a.q2 = p->qg2 + off; a.y2 = p->yg2 + off; }
    a.gtw = p->gtw; a.gtw_n = p->gtw_n;
    a.kv_elems = a.slices * p->vol;
    a.h_elems = (shared ? p->C : a.slices) * p->kvol;
    p->prof.begin(KID_FUSED2D, st);
    int c = launch_fused2d(a, p->log2p[2], p->dtype, st);
    p->prof.end(st);
    if (c < 0) return -1;
    *launches += c;
    return 0;
}

static int run_forward(hyenand_plan *p, const void *q, const void *k, const void *v, const void *h,
                       bool shared, void *y, cudaStream_t st, int *launches)
{
    int rc;
    if (p->path == PATH_FUSED2D)
        rc = forward_fused2d(p, q, k, v, h, shared, y, st, launches);
    else if (p->path == PATH_PLANES3D)
        rc = forward_planes3d(p, (const char *)q, (const char *)k, (const char *)v, (const char *)h, shared,
                              (char *)y, st, launches);
    else if (p->path == PATH_CT1D)
    {
        p->ct.r0 = p->r0; p->ct.r1 = p->r1;
        p->ct.dt_in = p->dt_in; p->ct.dt_out = p->dt_out; p->ct.dt_h = p->h_dtype;
        rc = ct1d_forward(&p->ct, q, k, v, h, shared, y, st, launches, &p->prof);
    }
    else
        rc = forward_generic(p, (const char *)q, (const char *)k, (const char *)v, (const char *)h, shared,
                             (char *)y, st, launches);
    if (rc == -2) return HYENAND_ERR_ALLOC;              // (message already recorded by the allocation)
    if (rc) return fail(HYENAND_ERR_CUDA, "internal launch dispatch failed");
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return fail(HYENAND_ERR_CUDA, "kernel launch failed: %s", cudaGetErrorString(e));
    return HYENAND_OK;
}

// y must not overlap an input (the kernels read the inputs while they write y)
static int check_overlap(const hyenand_plan *p, bool shared, const void *q, const void *k, const void *v, const void *h,
                         const void *y)
{
    const size_t es = elsize(p->dtype);
    const size_t nbytes = (size_t)p->B * p->C * p->vol * es;
    const size_t hbytes = (size_t)(shared ? 1 : p->B) * p->C * p->kvol * es;
    const char *yb = (const char *)y;
    const void *ins[4] = {q, k, v, h};
    for (int i = 0; i < 4; ++i) {
        const char *ib = (const char *)ins[i];
        const size_t ilen = i == 3 ? hbytes : nbytes;
        if (yb < ib + ilen && ib < yb + nbytes) return fail(HYENAND_ERR_INVALID_ARG, "y overlaps input %d", i);
    }
    return HYENAND_OK;
}

// a plan's workspace, streams and tensor maps belong to the device it was created on
static int check_device(const hyenand_plan *p)
{
    int cur = -1;
    if (cudaGetDevice(&cur) != cudaSuccess) return fail(HYENAND_ERR_CUDA, "cudaGetDevice failed");
    if (cur != p->device)
        return fail(HYENAND_ERR_INVALID_ARG, "the plan belongs to device %d but device %d is current", p->device, cur);
    return HYENAND_OK;
}

static int check_stride(hyenand_plan *p, long long hs, bool *shared)
{
    if (hs == 0) { *shared = true; return HYENAND_OK; }
    if (hs == (long long)p->C * p->kvol) { *shared = false; return HYENAND_OK; }
    return fail(HYENAND_ERR_INVALID_ARG, "h_batch_stride_elems must be 0 or C*K_1*..*K_N = %lld (got %lld)",
                (long long)p->C * p->kvol, hs);
}

extern "C" int hyenand_forward_ex(hyenand_plan *p, const void *q, const void *k, const void *v, const void *h,
                                  long long h_batch_stride_elems, void *y, void *cuda_stream)
{
    g_err[0] = 0;
    if (!p) return fail(HYENAND_ERR_INVALID_ARG, "plan is NULL");
    if (!q || !k || !v || !h || !y) return fail(HYENAND_ERR_INVALID_ARG, "q, k, v, h, y must be non-NULL");
    const void *ptrs[5] = {q, k, v, h, y};
    for (int i = 0; i < 5; ++i)
        if (((uintptr_t)ptrs[i]) & 15) return fail(HYENAND_ERR_INVALID_ARG, "pointer %d is not 16-byte aligned", i);
    bool shared = false;
    int e = check_stride(p, h_batch_stride_elems, &shared);
    if (!e) e = check_overlap(p, shared, q, k, v, h, y);
    if (!e) e = check_device(p);
    if (e) return e;
    {
        DbgScope d;
        const size_t nbytes = (size_t)p->B * p->C * p->vol * elsize(p->dtype);
        d.add(q, nbytes); d.add(k, nbytes); d.add(v, nbytes); d.add(y, nbytes);
        d.add(h, (size_t)(shared ? 1 : p->B) * p->C * p->kvol * elsize(p->dtype));
        d.add(p->allocs);
        d.commit();
    }
    int launches = 0;
    return run_forward(p, q, k, v, h, shared, y, (cudaStream_t)cuda_stream, &launches);
}

extern "C" int hyenand_forward(hyenand_plan *p, const void *q, const void *k, const void *v, const void *h,
                               void *y, void *cuda_stream)
{
    if (!p) { g_err[0] = 0; return fail(HYENAND_ERR_INVALID_ARG, "plan is NULL"); }
    return hyenand_forward_ex(p, q, k, v, h, (long long)p->C * p->kvol, y, cuda_stream);
}

extern "C" int hyenand_forward_host(hyenand_plan *p, const void *q, const void *k, const void *v, const void *h,
                                    long long h_batch_stride_elems, void *y, void *cuda_stream)
{
    g_err[0] = 0;
    if (!p) return fail(HYENAND_ERR_INVALID_ARG, "plan is NULL");
    if (!q || !k || !v || !h || !y) return fail(HYENAND_ERR_INVALID_ARG, "q, k, v, h, y must be non-NULL");
    bool shared = false;
    int e = check_stride(p, h_batch_stride_elems, &shared);
    if (!e) e = check_device(p);
    if (e) return e;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const size_t es = elsize(p->dtype);
    const size_t nbytes = (size_t)p->B * p->C * p->vol * es;
    const size_t hbytes = (size_t)(shared ? 1 : p->B) * p->C * p->kvol * es;
    const size_t want[5] = {nbytes, nbytes, nbytes, hbytes, nbytes};
    for (int i = 0; i < 5; ++i) {
        if (p->stage_bytes[i] < want[i]) {
            if (p->stage[i]) { cudaFree(p->stage[i]); p->ws_bytes -= p->stage_bytes[i]; p->stage[i] = nullptr; p->stage_bytes[i] = 0; }
            // staging copies of the caller's tensors: plain allocations, re-sized on demand (not workspace)
            cudaError_t ce = cudaMalloc(&p->stage[i], want[i] ? want[i] : 16);
            if (ce != cudaSuccess) {
                cudaGetLastError();
                p->stage[i] = nullptr;
                return fail(HYENAND_ERR_ALLOC, "cudaMalloc of %zu staging bytes failed: %s", want[i], cudaGetErrorString(ce));
            }
            p->ws_bytes += want[i];
            p->stage_bytes[i] = want[i];
        }
    }
    {
        DbgScope d;
        for (int i = 0; i < 5; ++i) d.add(p->stage[i], p->stage_bytes[i]);
        d.add(p->allocs);
        d.commit();
    }
    // Pipeline over groups of slices: the inputs of group g+1 travel to the device (copy-in stream) while group g
    // is computed (caller's stream) and the result of group g-1 travels back (copy-out stream).  A filter shared
    // over the batch goes first, whole.  With one group this is copy, compute, copy.
    if (!p->copy_in) {
        if (cudaStreamCreateWithFlags(&p->copy_in, cudaStreamNonBlocking) != cudaSuccess ||
            cudaStreamCreateWithFlags(&p->copy_out, cudaStreamNonBlocking) != cudaSuccess ||
            cudaEventCreateWithFlags(&p->ev_in[0], cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&p->ev_in[1], cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&p->ev_out, cudaEventDisableTiming) != cudaSuccess)
            return fail(HYENAND_ERR_CUDA, "pipeline streams: %s", cudaGetErrorString(cudaGetLastError()));
    }
    const long long S = (long long)p->B * p->C;
    const size_t sl = (size_t)p->vol * es, hsl = (size_t)p->kvol * es;       // bytes per slice
    long long groups = S < 8 ? S : 8;
    if (nbytes + hbytes < ((size_t)64 << 20)) groups = 1;                      // small problems: nothing to overlap
    const long long per = (S + groups - 1) / groups;
    int launches = 0;
    bool bad = false;
    // the copy-in stream starts after whatever the caller's stream holds (the staging buffers may still be read)
    bad |= cudaEventRecord(p->ev_out, st) != cudaSuccess || cudaStreamWaitEvent(p->copy_in, p->ev_out, 0) != cudaSuccess;
    if (shared) bad |= cudaMemcpyAsync(p->stage[3], h, hbytes, cudaMemcpyHostToDevice, p->copy_in) != cudaSuccess;
    int g = 0;
    for (long long s0 = 0; s0 < S && !bad; s0 += per, ++g) {
        const long long n = S - s0 < per ? S - s0 : per;
        const void *src[3] = {k, v, q};
        const int dsti[3] = {1, 2, 0};
        if (!shared)
            bad |= cudaMemcpyAsync((char *)p->stage[3] + s0 * hsl, (const char *)h + s0 * hsl, n * hsl, cudaMemcpyHostToDevice, p->copy_in) != cudaSuccess;
        for (int i = 0; i < 3; ++i)
            bad |= cudaMemcpyAsync((char *)p->stage[dsti[i]] + s0 * sl, (const char *)src[i] + s0 * sl, n * sl, cudaMemcpyHostToDevice, p->copy_in) != cudaSuccess;
        cudaEvent_t ev = p->ev_in[g & 1];
        // an event is reused every other group: by then the compute stream has long passed its previous wait
        bad |= cudaEventRecord(ev, p->copy_in) != cudaSuccess || cudaStreamWaitEvent(st, ev, 0) != cudaSuccess;
        if (bad) break;
        p->r0 = s0; p->r1 = s0 + n;
        e = run_forward(p, p->stage[0], p->stage[1], p->stage[2], p->stage[3], shared, p->stage[4], st, &launches);
        p->r0 = 0; p->r1 = S;
        if (e) return e;
        bad |= cudaEventRecord(p->ev_out, st) != cudaSuccess || cudaStreamWaitEvent(p->copy_out, p->ev_out, 0) != cudaSuccess;
        bad |= cudaMemcpyAsync((char *)y + s0 * sl, (char *)p->stage[4] + s0 * sl, n * sl, cudaMemcpyDeviceToHost, p->copy_out) != cudaSuccess;
    }
    if (bad) return fail(HYENAND_ERR_CUDA, "pipelined host copy failed: %s", cudaGetErrorString(cudaGetLastError()));
    cudaError_t ce = cudaStreamSynchronize(p->copy_out);
    if (ce == cudaSuccess) ce = cudaStreamSynchronize(p->copy_in);
    if (ce == cudaSuccess) ce = cudaStreamSynchronize(st);
    if (ce != cudaSuccess) return fail(HYENAND_ERR_CUDA, "stream synchronise failed: %s", cudaGetErrorString(ce));
    return HYENAND_OK;
}

extern "C" size_t hyenand_plan_workspace_bytes(const hyenand_plan *p) { return p ? p->ws_bytes : 0; }

extern "C" int hyenand_plan_fft_dims(const hyenand_plan *p, int *out_P)
{
    g_err[0] = 0;
    if (!p || !out_P) return fail(HYENAND_ERR_INVALID_ARG, "NULL argument");
    for (int a = 0; a < p->ndim; ++a) out_P[a] = p->P[3 - p->ndim + a];
    return HYENAND_OK;
}

extern "C" int hyenand_plan_launches(const hyenand_plan *p, int h_shared)
{
    if (!p) return 0;
    if (p->path == PATH_CT1D) return ct1d_launches(&p->ct, h_shared != 0);
    const long long S = (long long)p->B * p->C;
    const long long chunks = (S + p->slices_per_chunk - 1) / p->slices_per_chunk;
    const int three = p->P[0] > 1;
    if (p->path == PATH_FUSED2D) return 1;
    if (p->path == PATH_PLANES3D) return (int)(h_shared ? 1 + chunks * 3 : chunks * 4);
    const int filt = 1 + three, body = 3 + 2 * three;
    return (int)(h_shared ? filt + chunks * body : chunks * (filt + body));
}

extern "C" int hyenand_plan_groups(const hyenand_plan *p, long long *slices_per_group, int *lanes)
{
    g_err[0] = 0;
    if (!p) return fail(HYENAND_ERR_INVALID_ARG, "plan is NULL");
    if (slices_per_group) *slices_per_group = p->path == PATH_CT1D ? p->ct.slices_per_chunk : p->path == PATH_FUSED2D ? (long long)p->B * p->C : p->slices_per_chunk;
    if (lanes) *lanes = p->path == PATH_CT1D || p->path == PATH_FUSED2D ? 1 : p->n_lanes;
    return HYENAND_OK;
}

extern "C" const char *hyenand_plan_path(const hyenand_plan *p)
{
    if (!p) return "";
    return p->path == PATH_CT1D ? "ct1d" : p->path == PATH_PLANES3D ? "planes3d"
         : p->path == PATH_FUSED2D ? "fused2d" : "nd_generic";
}

// ---- per-kernel accounting (reporting only) ---------------------------------------------

const char *const hn::kKernelNames[KID_COUNT] = {
    "rows_fwd(h)", "axis_fwd(h)", "rows_fwd(k*v)", "axis_fwd(k*v)", "axis_core", "axis_inv", "rows_inv",
    "ct_cols_fwd(h)", "ct_cols_fwd(k*v)", "ct_core", "ct_cols_inv", "plane_fwd(h)", "plane_fwd(k*v)", "plane_inv", "fused2d", "ct_hspec"};

static double fft_flops(double lines, int log2n) { return lines * 5.0 * ldexp(1.0, log2n) * log2n; }

extern "C" int hyenand_plan_kernel_count(const hyenand_plan *p) { return p ? KID_COUNT : 0; }

extern "C" int hyenand_plan_kernel_info(const hyenand_plan *p, int kid, int h_shared, const char **name,
                                        double *launches, double *bytes, double *flops)
{
    g_err[0] = 0;
    if (!p || kid < 0 || kid >= KID_COUNT || !name || !launches || !bytes || !flops)
        return fail(HYENAND_ERR_INVALID_ARG, "bad argument");
    *name = kKernelNames[kid];
    *launches = *bytes = *flops = 0.0;
    const double S = (double)p->B * p->C, Sh = h_shared ? p->C : S;
    const double es = (double)elsize(p->dtype), c8 = 8.0;
    if (p->path == PATH_CT1D) {
        const Ct1dPlan &c = p->ct;
        const double P1 = ldexp(1.0, c.log2p1), P2 = ldexp(1.0, c.log2p2), F1 = P1 / 2 + 1;
        const double chunks = ceil(S / (double)c.slices_per_chunk);
        switch (kid) {
        case KID_CT_COLS_H:
            *launches = h_shared ? 1 : chunks; *bytes = Sh * (c.K * es + F1 * P2 * c8);
            *flops = fft_flops(Sh * P2 / 2, c.log2p1); break;
        case KID_CT_COLS_U:
            *launches = chunks; *bytes = S * (2 * c.L * es + F1 * P2 * c8);
            *flops = fft_flops(S * P2 / 2, c.log2p1); break;
        case KID_CT_CORE:
            if (ct1d_uses_w(&c)) {
                *launches = chunks; *bytes = S * 3 * F1 * P2 * c8;
                *flops = 2 * fft_flops(S * F1, c.log2p2) + 12.0 * S * F1 * P2;
            } else {
                *launches = chunks; *bytes = S * 3 * F1 * P2 * c8;
                *flops = 3 * fft_flops(S * F1, c.log2p2) + 12.0 * S * F1 * P2;
            }
            break;
        case KID_CT_HSPEC:
            if (ct1d_uses_w(&c)) {
                *launches = h_shared ? 1 : chunks; *bytes = Sh * 2 * F1 * P2 * c8;
                *flops = fft_flops(Sh * F1, c.log2p2);
            }
            break;
        case KID_CT_COLS_INV:
            *launches = chunks; *bytes = S * (F1 * P2 * c8 + 2 * c.L * es);
            *flops = fft_flops(S * P2 / 2, c.log2p1); break;
        default: break;
        }
        return HYENAND_OK;
    }
    const bool three = p->P[0] > 1;
    const double chunks = ceil(S / (double)p->slices_per_chunk);
    if (p->path == PATH_FUSED2D) {
        if (kid == KID_FUSED2D) {
            const double PP = p->P[2], XHd = p->XH;
            *launches = 1;
            *bytes = 4.0 * S * p->vol * es + Sh * (double)p->kvol * es;
            *flops = fft_flops(S * PP / 2.0, p->log2p[2]) + 2.0 * fft_flops(S * p->L[1] / 2.0, p->log2p[2])
                   + 3.0 * fft_flops(S * XHd, p->log2p[1]) + 12.0 * S * XHd * PP;
        }
        return HYENAND_OK;
    }
    if (p->path == PATH_PLANES3D) {
        const double PY = p->P[1], nc = (double)p->XH * PY, Lz = p->L[0], Kz = p->K[0];
        const double rowsU = p->L[1] / 2.0, colsU = PY / 2.0;
        switch (kid) {
        case KID_PLANE_H:
            *launches = h_shared ? 1 : chunks; *bytes = Sh * ((double)p->kvol * es + Kz * nc * c8);
            *flops = fft_flops(Sh * Kz * PY / 2.0, p->log2p[2]) + fft_flops(Sh * Kz * p->P[2] / 2.0, p->log2p[1]); break;
        case KID_PLANE_U:
            *launches = chunks; *bytes = S * (2.0 * p->vol * es + Lz * nc * c8);
            *flops = fft_flops(S * Lz * rowsU, p->log2p[2]) + fft_flops(S * Lz * colsU, p->log2p[1]); break;
        case KID_CORE:
            *launches = chunks; *bytes = S * nc * c8 * (2.0 * Lz + Kz);
            *flops = 3 * fft_flops(S * nc, p->log2p[0]) + 12.0 * S * nc * p->P[0]; break;
        case KID_PLANE_INV:
            *launches = chunks; *bytes = S * (Lz * nc * c8 + 2.0 * p->vol * es);
            *flops = fft_flops(S * Lz * rowsU, p->log2p[2]) + fft_flops(S * Lz * colsU, p->log2p[1]); break;
        default: break;
        }
        return HYENAND_OK;
    }
    const double XH = p->XP, L0 = p->L[0], L1 = p->L[1], L2 = p->L[2], K0 = p->K[0], K1 = p->K[1], P1 = p->P[1];
    const int ax = three ? 0 : 1;
    const double inner = three ? P1 * XH : XH;
    switch (kid) {
    case KID_ROWS_H:
        *launches = h_shared ? 1 : chunks; *bytes = Sh * ((double)p->kvol * es + K0 * K1 * XH * c8);
        *flops = fft_flops(Sh * K0 * K1 / 2, p->log2p[2]); break;
    case KID_AXIS_H:
        if (three) { *launches = h_shared ? 1 : chunks; *bytes = Sh * K0 * XH * c8 * (K1 + P1);
                     *flops = fft_flops(Sh * K0 * XH, p->log2p[1]); }
        break;
    case KID_ROWS_U:
        *launches = chunks; *bytes = S * (2.0 * p->vol * es + L0 * L1 * XH * c8);
        *flops = fft_flops(S * L0 * L1 / 2, p->log2p[2]); break;
    case KID_AXIS_U:
        if (three) { *launches = chunks; *bytes = S * L0 * XH * c8 * (L1 + P1);
                     *flops = fft_flops(S * L0 * XH, p->log2p[1]); }
        break;
    case KID_CORE:
        *launches = chunks; *bytes = S * inner * c8 * (2.0 * p->L[ax] + p->K[ax]);
        *flops = 3 * fft_flops(S * inner, p->log2p[ax]) + 12.0 * S * inner * p->P[ax]; break;
    case KID_AXIS_INV:
        if (three) { *launches = chunks; *bytes = S * L0 * XH * c8 * (L1 + P1);
                     *flops = fft_flops(S * L0 * XH, p->log2p[1]); }
        break;
    case KID_ROWS_INV:
        *launches = chunks; *bytes = S * (L0 * L1 * XH * c8 + 2.0 * p->vol * es);
        *flops = fft_flops(S * L0 * L1 / 2, p->log2p[2]); break;
    default: break;
    }
    (void)L2;
    return HYENAND_OK;
}

extern "C" int hyenand_plan_set_timing(hyenand_plan *p, int enable)
{
    g_err[0] = 0;
    if (!p) return fail(HYENAND_ERR_INVALID_ARG, "plan is NULL");
    p->prof.on = enable != 0;
    p->serial_timing = enable == 2;
    p->prof.reset();
    return HYENAND_OK;
}

extern "C" int hyenand_plan_kernel_time(hyenand_plan *p, int kid, double *total_ms, double *launches)
{
    g_err[0] = 0;
    if (!p || kid < 0 || kid >= KID_COUNT || !total_ms || !launches) return fail(HYENAND_ERR_INVALID_ARG, "bad argument");
    p->prof.collect();
    *total_ms = p->prof.ms[kid];
    *launches = (double)p->prof.launches[kid];
    return HYENAND_OK;
}

// ---- the full HyenaND operator (Eq. 2): pointwise stages around the long convolution -----------------
//
// The long convolution runs on an fp32 plan whatever the I/O type, so that nothing between the first read of
// q, k, v and the final store of y is rounded below fp32: the pre-stage writes its three results in fp32, the
// kernel h is widened once per call when the I/O type is bf16, and the post-stage reads the gated convolution
// in fp32.  Batches are worked off in groups of batch entries that bound the fp32 scratch.

struct hyenand_mixer {
    hyenand_plan *plan;               // fp32 plan over nb batch entries
    int B, C, dtype, nb;              // nb: batch entries per pass
    long long L, kvol;
    float eps;
    float *qz, *kz, *vz, *oz, *h32;   // scratch, fp32 (h32: widened bf16 taps, only where the inner plan cannot read them itself)
    bool h_native;                    // the inner plan reads the taps in the caller's element type
    GuardedAllocs allocs;
    int device;
};

extern "C" void hyenand_mixer_destroy(hyenand_mixer *m)
{
    if (!m) return;
    int cur = 0;
    cudaGetDevice(&cur);
    if (cur != m->device) cudaSetDevice(m->device);
    hyenand_destroy_plan(m->plan);
    guarded_free_all(&m->allocs);
    if (cur != m->device) cudaSetDevice(cur);
    delete m;
}

extern "C" hyenand_mixer *hyenand_mixer_create(int ndim, const int *dims, int B, int C, int mode, int dtype, float eps)
{
    g_err[0] = 0;
    if (dtype != HYENAND_F32 && dtype != HYENAND_BF16) { fail(HYENAND_ERR_INVALID_ARG, "unknown dtype %d", dtype); return nullptr; }
    if (!(eps >= 0.f)) { fail(HYENAND_ERR_INVALID_ARG, "eps must be >= 0"); return nullptr; }
    if (ndim < 1 || ndim > 3 || !dims || B < 1 || C < 1) { fail(HYENAND_ERR_INVALID_ARG, "bad geometry"); return nullptr; }
    long long L = 1;
    for (int a = 0; a < ndim; ++a) {
        if (dims[a] < 1) { fail(HYENAND_ERR_INVALID_ARG, "dims[%d] = %d must be >= 1", a, dims[a]); return nullptr; }
        L *= dims[a];
    }
    // batch entries per pass: four fp32 tensors of nb*C*L elements, at most 2 GiB together
    long long nb = (2ll << 30) / (16ll * C * L);
    if (const char *e = getenv("HYENAND_MIXER_MAX_BATCH")) { const long long v = atoll(e); if (v > 0 && v < nb) nb = v; }   // development aid
    if (nb < 1) nb = 1;
    if (nb > B) nb = B;
    hyenand_plan *plan = hyenand_create_plan_mode(ndim, dims, (int)nb, C, mode, HYENAND_F32);
    if (!plan) return nullptr;
    hyenand_mixer *m = new hyenand_mixer();
    memset(m, 0, sizeof(*m));
    m->plan = plan; m->B = B; m->C = C; m->dtype = dtype; m->nb = (int)nb; m->L = L; m->kvol = plan->kvol; m->eps = eps;
    m->device = plan->device;
    m->h_native = plan_set_filter_dtype(plan, dtype);      // else bf16 taps are widened into h32 first
    const size_t n = (size_t)nb * C * L * sizeof(float);
    cudaError_t e = guarded_alloc(&m->allocs, (void **)&m->qz, n);
    if (e == cudaSuccess) e = guarded_alloc(&m->allocs, (void **)&m->kz, n);
    if (e == cudaSuccess) e = guarded_alloc(&m->allocs, (void **)&m->vz, n);
    if (e == cudaSuccess) e = guarded_alloc(&m->allocs, (void **)&m->oz, n);
    if (e == cudaSuccess && dtype == HYENAND_BF16 && !m->h_native)
        e = guarded_alloc(&m->allocs, (void **)&m->h32, (size_t)nb * C * m->kvol * sizeof(float));
    if (e != cudaSuccess) {
        cudaGetLastError();
        fail(HYENAND_ERR_ALLOC, "scratch of the pointwise stages: %s", cudaGetErrorString(e));
        hyenand_mixer_destroy(m);
        return nullptr;
    }
    return m;
}

extern "C" int hyenand_mixer_forward(hyenand_mixer *m, const void *q, const void *k, const void *v, const void *h,
                                     long long h_batch_stride_elems, const float *g_in, const float *g_out, void *y,
                                     void *cuda_stream)
{
    g_err[0] = 0;
    if (!m) return fail(HYENAND_ERR_INVALID_ARG, "mixer is NULL");
    if (!q || !k || !v || !h || !y || !g_in || !g_out) return fail(HYENAND_ERR_INVALID_ARG, "q, k, v, h, g_in, g_out, y must be non-NULL");
    const void *ptrs[5] = {q, k, v, h, y};
    for (int i = 0; i < 5; ++i)
        if (((uintptr_t)ptrs[i]) & 15) return fail(HYENAND_ERR_INVALID_ARG, "pointer %d is not 16-byte aligned", i);
    hyenand_plan *p = m->plan;
    bool shared = false;
    int e = check_stride(p, h_batch_stride_elems, &shared);
    if (!e) e = check_device(p);
    if (e) return e;
    const size_t es = elsize(m->dtype);
    {
        // y must not overlap an input (geometry of the whole batch, in the I/O type)
        const size_t nbytes = (size_t)m->B * m->C * m->L * es, hbytes = (size_t)(shared ? 1 : m->B) * m->C * m->kvol * es;
        const char *yb = (const char *)y;
        const void *ins[4] = {q, k, v, h};
        for (int i = 0; i < 4; ++i) {
            const char *ib = (const char *)ins[i];
            const size_t ilen = i == 3 ? hbytes : nbytes;
            if (yb < ib + ilen && ib < yb + nbytes) return fail(HYENAND_ERR_INVALID_ARG, "y overlaps input %d", i);
        }
    }
    {
        DbgScope d;
        const size_t nbytes = (size_t)m->B * m->C * m->L * es;
        d.add(q, nbytes); d.add(k, nbytes); d.add(v, nbytes); d.add(y, nbytes);
        d.add(h, (size_t)(shared ? 1 : m->B) * m->C * m->kvol * es);
        d.add(g_in, (size_t)m->C * sizeof(float)); d.add(g_out, (size_t)m->C * sizeof(float));
        d.add(m->allocs); d.add(p->allocs);
        d.commit();
    }
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const size_t slab = (size_t)m->C * m->L;                        // elements per batch entry
    const bool widen_h = m->dtype == HYENAND_BF16 && !m->h_native;
    const float *hf = (const float *)h;
    if (widen_h && shared) {
        launch_widen(h, m->dtype, (long long)m->C * m->kvol, m->h32, st);
        hf = m->h32;
    }
    for (int b0 = 0; b0 < m->B; b0 += m->nb) {
        const int n = m->B - b0 < m->nb ? m->B - b0 : m->nb;
        const char *qb = (const char *)q + (size_t)b0 * slab * es, *kb = (const char *)k + (size_t)b0 * slab * es,
                   *vb = (const char *)v + (size_t)b0 * slab * es;
        launch_mixer_pre(qb, kb, vb, g_in, m->eps, m->dtype, n, m->C, m->L, m->qz, m->kz, m->vz, st);
        const float *hb = hf;
        if (!shared) {
            if (widen_h) {
                launch_widen((const char *)h + (size_t)b0 * m->C * m->kvol * es, m->dtype, (long long)n * m->C * m->kvol, m->h32, st);
                hb = m->h32;
            } else {
                hb = (const float *)((const char *)h + (size_t)b0 * m->C * m->kvol * es);      // taps in the caller's type
            }
        }
        int launches = 0;
        p->r0 = 0; p->r1 = (long long)n * m->C;
        e = run_forward(p, m->qz, m->kz, m->vz, hb, shared, m->oz, st, &launches);
        p->r0 = 0; p->r1 = (long long)p->B * p->C;
        if (e) return e;
        launch_mixer_post(m->oz, g_out, m->eps, m->dtype, n, m->C, m->L, (char *)y + (size_t)b0 * slab * es, st);
    }
    cudaError_t ce = cudaGetLastError();
    if (ce != cudaSuccess) return fail(HYENAND_ERR_CUDA, "kernel launch failed: %s", cudaGetErrorString(ce));
    return HYENAND_OK;
}

extern "C" hyenand_plan *hyenand_mixer_plan(hyenand_mixer *m) { return m ? m->plan : nullptr; }

extern "C" long long hyenand_mixer_guard_damage(hyenand_mixer *m)
{
    g_err[0] = 0;
    if (!m) { fail(HYENAND_ERR_INVALID_ARG, "mixer is NULL"); return -1; }
    const long long a = guard_damage(&m->allocs), b = guard_damage(&m->plan->allocs);
    return (a < 0 || b < 0) ? -1 : a + b;
}

// ---- backward pass ----------------------------------------------------------------------------------------
//
// Forward: y = q * w, w = h conv u, u = k * v.  With g = dy * q:
//     dq = dy * w                         one forward with the outer gate dy
//     du = h' conv g, h'[d] = h[-d]       one forward with the kernel re-indexed to the opposite displacement
//     dk = du * v, dv = du * k
//     dh[d] = sum_i g_i u_{i-d}           a correlation of two grid signals whose result lives on the TAP grid:
//         - transforms up to 8192 points per axis: one circular convolution on the padded grid P (which holds every
//           displacement without wrap-around) of the zero-padded g with the zero-padded u at the opposite
//           displacement; the taps are read back from the ring;
//         - circular operators: the same on the grid itself;
//         - long 1-D: the causal forward applied to reversed signals (one call per sign of the displacement).
// Everything runs on fp32 plans and fp32 scratch (bf16 inputs are widened once), each gradient is rounded once, at
// its final store.  Batches are worked off in groups of batch entries, the dh correlation in groups of slices.

struct hyenand_grad {
    int ndim, B, C, mode, dtype, device;
    int dims[3];
    int L[3], K[3], P[3];             // internal 3-axis form
    long long vol, kvol, pvol, kopp;  // elements per slice: grid, taps, padded ring, taps of the opposite kernel
    bool long1d;
    bool h_native;                    // bf16 I/O: the forwards for dq and du read bf16 taps themselves (no widened kernel)
    bool pair;                        // dq and du come out of one pass over the groups (one filter spectrum serves both)
    bool ct_native;                   // long causal 1-D grid with bf16 I/O whose kernels take bf16 rows: k, v, dy, q, h are read as
                                      // they are, dq leaves its forward as bf16 (only the fp32 intermediates have scratch)
    bool two_gate;                    // fused 2-D path, linear mode: the plan runs in the caller's element type; dq is a forward
                                      // gated by dy, dk and dv are the two results of one forward gated by v and by k
    bool native;                      // bf16 I/O on the multi-kernel paths and with two_gate: every kernel reads the caller's bf16 tensors itself and
                                      // dq leaves its pass as bf16 (no widened copies of q, k, v, dy)
    int nb;                           // batch entries per pass
    long long ns;                     // slices per pass of the dh correlation (0: not on that path)
    hyenand_plan *main, *adj, *caus;
    float *q32, *k32, *v32, *dy32, *ones, *t32, *h32, *hopp;      // per pass of nb entries
    float2 *cga, *cgb, *cua, *cub, *cwc, *cwd;                   // dh correlation: spectra of ns slices (see corr_dh)
    float *aux;                       // nb*C slices: reversed signals of the long 1-D path
    float *dhs;                       // nb*C slices of taps: per-slice kernel gradients before the sum over the batch
    float *dh32;                      // accumulated kernel gradient (shared kernel: [C][kvol]; else [nb*C][kvol])
    GuardedAllocs allocs;
};

extern "C" void hyenand_backward_destroy(hyenand_grad *g)
{
    if (!g) return;
    int cur = 0;
    cudaGetDevice(&cur);
    if (cur != g->device) cudaSetDevice(g->device);
    if (g->adj && g->adj != g->main) hyenand_destroy_plan(g->adj);
    if (g->caus && g->caus != g->main) hyenand_destroy_plan(g->caus);
    hyenand_destroy_plan(g->main);
    guarded_free_all(&g->allocs);
    if (cur != g->device) cudaSetDevice(cur);
    delete g;
}

// ---- dh as a correlation on the general N-D kernels --------------------------------------------------------------
// dh[d + L-1] = sum_t g[t] u[t - d] with g = dy q and u = k v is the full linear convolution of g with u reversed
// along every axis: both operands have L points per axis (the zero half of their padded lines is pruned from the
// forward transforms, like the k*v side of a forward), all 2L-1 outputs per axis are kept.  The stages are those of
// the general path -- rows, [middle axis in 3-D], fused core along the last transformed axis, [middle axis back],
// rows back -- on spectra of this handle's own (nothing padded is ever materialised; the first version ran a
// circular convolution over padded copies of all three tensors, 55 of the 71 ms of a volume3d backward).
struct CorrGeo {
    long long rows_in;      // [L0][L1][XP]   row spectra of an operand
    long long mid;          // [L0][P1][XP]   after the middle axis (3-D only)
    long long core_out;     // [K0][P1][XP]   (3-D) or [K1][XP] (1-D, 2-D): after the core
    long long inv_out;      // [K0][K1][XP]   (3-D only): after the middle axis back
};

static CorrGeo corr_geo(const hyenand_grad *g)
{
    const hyenand_plan *p = g->main;
    const long long XP = p->XP;
    const long long K0 = 2ll * g->L[0] - 1, K1 = 2ll * g->L[1] - 1;
    const bool three = g->P[0] > 1;
    CorrGeo c{};
    c.rows_in = (long long)g->L[0] * g->L[1] * XP;
    c.mid = three ? (long long)g->L[0] * g->P[1] * XP : 0;
    c.core_out = three ? K0 * g->P[1] * XP : K1 * XP;
    c.inv_out = three ? K0 * K1 * XP : 0;
    return c;
}

static long long corr_slice_elems(const hyenand_grad *g)
{
    const CorrGeo c = corr_geo(g);
    return 2 * c.rows_in + 2 * c.mid + c.core_out + c.inv_out;
}

// m slices: gy, gq (elements of g_dtype; their product is g), ur (u reversed, fp32) -> out [m][2L0-1][2L1-1][2L2-1],
// elements of type out_dtype
static int corr_dh(hyenand_grad *g, long long m, const void *gy, const void *gq, int g_dtype, const float *ur, void *out,
                   int out_dtype, cudaStream_t st)
{
    hyenand_plan *p = g->main;                          // geometry, twiddles, switches
    const int *L = g->L, *P = g->P;
    const int K0 = 2 * L[0] - 1, K1 = 2 * L[1] - 1, K2 = 2 * L[2] - 1;
    const bool three = P[0] > 1;
    const int XP = p->XP;
    int c = 0;
    auto rows = [&](const void *a, const void *b, int dt, float2 *dst) {
        RowsArgs r{};
        r.a = a; r.b = b; r.out = dst; r.pitch = XP;
        r.rows = m * L[0] * L[1]; r.len = L[2]; r.shift = 0; r.log2p = p->log2p[2];
        r.prune_in = p->P[2] >= 2; r.full_in = 0; r.gtw = p->gtw; r.gtw_n = p->gtw_n;
        const bool roww = rows_w_supported(r.log2p) && !p->sw.generic_rows;
        return roww ? launch_rows_fwd_w(r, dt, st) : launch_rows_fwd(r, dt, st);
    };
    auto middle = [&](const float2 *src, float2 *dst) {
        AxisArgs a{};
        a.in = src; a.out = dst;
        a.n_outer = m * L[0];
        a.in_outer = (long long)L[1] * XP; a.out_outer = (long long)P[1] * XP;
        a.nc = XP; a.n_in = L[1]; a.n_out = P[1]; a.shift = 0;
        a.log2p = p->log2p[1]; a.prune_in = P[1] >= 2;
        a.gtw = p->gtw; a.gtw_n = p->gtw_n;
        return launch_axis_any(p->sw, a, AXIS_FWD, st);
    };
    if ((c = rows(gy, gq, g_dtype, g->cga)) < 0) return fail(HYENAND_ERR_CUDA, "internal launch dispatch failed");
    if ((c = rows(ur, nullptr, HYENAND_F32, g->cua)) < 0) return fail(HYENAND_ERR_CUDA, "internal launch dispatch failed");
    if (three) {
        if ((c = middle(g->cga, g->cgb)) < 0 || (c = middle(g->cua, g->cub)) < 0)
            return fail(HYENAND_ERR_CUDA, "internal launch dispatch failed");
    }
    {
        const int ax = three ? 0 : 1;                   // core axis
        const int Kax = three ? K0 : K1;
        const long long inner = three ? (long long)P[1] * XP : XP;
        AxisArgs a{};
        a.in = three ? g->cgb : g->cga; a.out = g->cwc;
        a.n_outer = m;
        a.in_outer = (long long)L[ax] * inner; a.out_outer = (long long)Kax * inner;
        a.nc = (int)inner; a.n_in = L[ax]; a.n_out = Kax; a.shift = 0;
        a.log2p = p->log2p[ax]; a.prune_in = 0; a.full = 1;
        a.h = three ? g->cub : g->cua; a.h_outer = (long long)L[ax] * inner; a.h_n_in = L[ax]; a.h_shift = 0;
        a.h_mod = 0; a.h_off = 0;
        a.scale = (float)(1.0 / ((double)P[0] * P[1] * P[2]));
        a.gtw = p->gtw; a.gtw_n = p->gtw_n;
        c = (core_w_supported(a.log2p) && !p->sw.generic_core) ? launch_core_w(a, st) : launch_axis(a, AXIS_CORE, st);
        if (c < 0) return fail(HYENAND_ERR_CUDA, "internal launch dispatch failed");
    }
    if (three) {
        AxisArgs a{};
        a.in = g->cwc; a.out = g->cwd;
        a.n_outer = m * K0;
        a.in_outer = (long long)P[1] * XP; a.out_outer = (long long)K1 * XP;
        a.nc = XP; a.n_in = P[1]; a.n_out = K1; a.shift = 0;
        a.log2p = p->log2p[1]; a.prune_in = 0; a.full = 1;
        a.gtw = p->gtw; a.gtw_n = p->gtw_n;
        if ((c = launch_axis_any(p->sw, a, AXIS_INV, st)) < 0) return fail(HYENAND_ERR_CUDA, "internal launch dispatch failed");
    }
    {
        RowsInvArgs ri{};
        ri.in = three ? g->cwd : g->cwc; ri.pitch = XP; ri.q = nullptr; ri.y = out;
        ri.rows = m * K0 * K1; ri.len = K2; ri.log2p = p->log2p[2];
        ri.gtw = p->gtw; ri.gtw_n = p->gtw_n; ri.full_out = 1;
        const bool roww = rows_w_supported(ri.log2p) && !p->sw.generic_rows;
        c = roww ? launch_rows_inv_w(ri, out_dtype, st) : launch_rows_inv(ri, out_dtype, st);
        if (c < 0) return fail(HYENAND_ERR_CUDA, "internal launch dispatch failed");
    }
    return HYENAND_OK;
}

extern "C" hyenand_grad *hyenand_backward_create(int ndim, const int *dims, int B, int C, int mode, int dtype)
{
    g_err[0] = 0;
    if (dtype != HYENAND_F32 && dtype != HYENAND_BF16) { fail(HYENAND_ERR_INVALID_ARG, "unknown dtype %d", dtype); return nullptr; }
    if (ndim < 1 || ndim > 3 || !dims || B < 1 || C < 1) { fail(HYENAND_ERR_INVALID_ARG, "bad geometry"); return nullptr; }
    for (int a = 0; a < ndim; ++a)
        if (dims[a] < 1) { fail(HYENAND_ERR_INVALID_ARG, "dims[%d] = %d must be >= 1", a, dims[a]); return nullptr; }
    hyenand_grad *g = new hyenand_grad();
    memset(g, 0, sizeof(*g));
    cudaGetDevice(&g->device);
    g->ndim = ndim; g->B = B; g->C = C; g->mode = mode; g->dtype = dtype;
    g->vol = g->kvol = g->pvol = 1;
    for (int a = 0; a < 3; ++a) { g->L[a] = g->K[a] = g->P[a] = 1; }
    bool ring_ok = true;
    for (int a = 0; a < ndim; ++a) {
        const int ia = 3 - ndim + a;
        g->dims[a] = dims[a];
        g->L[ia] = dims[a];
        g->K[ia] = mode == HYENAND_MODE_LINEAR ? 2 * dims[a] - 1 : dims[a];
        g->P[ia] = mode == HYENAND_MODE_CIRCULAR ? dims[a] : 1 << next_pow2_log(2 * dims[a] - 1);
        if (g->P[ia] > (1 << kMaxLineLog2)) ring_ok = false;
        g->vol *= dims[a]; g->kvol *= g->K[ia]; g->pvol *= g->P[ia];
    }
    g->kopp = mode == HYENAND_MODE_CAUSAL ? 2ll * g->L[2] - 1 : g->kvol;
    g->long1d = !ring_ok;
    if (g->long1d && (ndim != 1 || mode == HYENAND_MODE_CIRCULAR)) {
        fail(HYENAND_ERR_UNSUPPORTED, "a padded axis exceeds %d points (only 1-D linear and causal grids may)", 1 << kMaxLineLog2);
        delete g; return nullptr;
    }
    // batch entries per pass: nine fp32 tensors of nb*C*vol elements (+ kernels) within about 4 GiB
    long long nb = (4ll << 30) / (4ll * C * (8 * g->vol + g->kopp + 3 * g->kvol));
    if (const char *e = getenv("HYENAND_BACKWARD_MAX_BATCH")) { const long long v = atoll(e); if (v > 0 && v < nb) nb = v; }   // development aid
    if (nb < 1) nb = 1;
    if (nb > B) nb = B;
    g->nb = (int)nb;
    const long long S = nb * C;
    g->main = hyenand_create_plan_mode(ndim, dims, (int)nb, C, mode, HYENAND_F32);
    if (!g->main) { delete g; return nullptr; }
    g->two_gate = g->main->path == PATH_FUSED2D && mode == HYENAND_MODE_LINEAR;
    if (g->two_gate && dtype != HYENAND_F32) {
        hyenand_destroy_plan(g->main);
        g->main = hyenand_create_plan_mode(ndim, dims, (int)nb, C, mode, dtype);
        if (!g->main) { delete g; return nullptr; }
    }
    g->adj = g->main;
    g->pair = g->main->path == PATH_PLANES3D || g->main->path == PATH_ND_GENERIC;
    // (a long causal 1-D grid gets du from the causal plan and reversed signals, see hyenand_backward)
    if (mode == HYENAND_MODE_CAUSAL && !g->pair && !g->long1d) {
        g->adj = hyenand_create_plan_mode(ndim, dims, (int)nb, C, HYENAND_MODE_LINEAR, HYENAND_F32);
        if (!g->adj) { g->adj = g->main; hyenand_backward_destroy(g); return nullptr; }
    }
    if (g->long1d) {
        g->caus = g->main;
        if (mode != HYENAND_MODE_CAUSAL) {
            g->caus = hyenand_create_plan_mode(ndim, dims, (int)nb, C, HYENAND_MODE_CAUSAL, HYENAND_F32);
            if (!g->caus) { hyenand_backward_destroy(g); return nullptr; }
        }
    } else if (mode != HYENAND_MODE_CIRCULAR) {
        // dh correlation: the spectra of ns slices within about 2 GiB
        long long ns = (2ll << 30) / (8ll * corr_slice_elems(g));
        if (const char *e = getenv("HYENAND_BACKWARD_RING_SLICES")) { const long long v = atoll(e); if (v > 0 && v < ns) ns = v; }   // development aid
        if (ns < 1) ns = 1;
        if (ns > S) ns = S;
        g->ns = ns;
    }
    const bool widen = dtype == HYENAND_BF16;
    auto reads_bf16 = [](const hyenand_plan *q) { return q->path == PATH_PLANES3D || q->path == PATH_ND_GENERIC; };
    g->ct_native = widen && g->long1d && mode == HYENAND_MODE_CAUSAL && g->main->path == PATH_CT1D &&
                   ct1d_takes_dtype(&g->main->ct, HYENAND_BF16);
    g->h_native = widen && ((reads_bf16(g->main) && reads_bf16(g->adj)) || g->two_gate || g->ct_native);
    g->native = widen && ((g->pair && mode != HYENAND_MODE_CIRCULAR && !g->long1d) || g->two_gate || g->ct_native);
    cudaError_t e = cudaSuccess;
    auto get = [&](float **ptr, long long elems) {
        if (e == cudaSuccess) e = guarded_alloc(&g->allocs, (void **)ptr, (size_t)elems * sizeof(float));
    };
    if (widen && !g->native) { get(&g->q32, S * g->vol); get(&g->k32, S * g->vol); get(&g->v32, S * g->vol); get(&g->dy32, S * g->vol); }
    if (widen && !g->h_native) get(&g->h32, S * g->kvol);
    if (!g->native || g->ct_native) { get(&g->ones, S * g->vol); get(&g->t32, S * g->vol); }
    get(&g->hopp, S * g->kopp);
    get(&g->aux, S * g->vol); get(&g->dhs, S * g->kvol); get(&g->dh32, S * g->kvol);
    if (g->ns) {
        const CorrGeo c = corr_geo(g);
        auto get2 = [&](float2 **ptr, long long elems) { if (elems) get((float **)ptr, 2 * elems * g->ns); };
        get2(&g->cga, c.rows_in); get2(&g->cua, c.rows_in); get2(&g->cgb, c.mid); get2(&g->cub, c.mid);
        get2(&g->cwc, c.core_out); get2(&g->cwd, c.inv_out);
    }
    if (e != cudaSuccess) {
        cudaGetLastError();
        fail(HYENAND_ERR_ALLOC, "scratch of the backward pass: %s", cudaGetErrorString(e));
        hyenand_backward_destroy(g);
        return nullptr;
    }
    { DbgScope d; d.add(g->allocs); d.commit(); }
    if (g->ones) launch_fill(g->ones, 1.f, S * g->vol, 0);
    if (cudaDeviceSynchronize() != cudaSuccess) {
        fail(HYENAND_ERR_CUDA, "filling the constant tensors failed: %s", cudaGetErrorString(cudaGetLastError()));
        hyenand_backward_destroy(g);
        return nullptr;
    }
    return g;
}

// one forward of `n` slices on an inner fp32 plan (a plan of more slices runs the first n)
static int grad_forward(hyenand_plan *p, long long n, const float *q, const float *k, const float *v, const void *h,
                        bool shared, float *y, cudaStream_t st, int h_dtype = HYENAND_F32, int dt_in = -1, int dt_out = -1)
{
    int launches = 0;
    if (!plan_set_filter_dtype(p, h_dtype)) return fail(HYENAND_ERR_UNSUPPORTED, "filter element type on this path");
    if (dt_in >= 0) p->dt_in = dt_in;                    // (paths that take an element type per stage; reset below)
    if (dt_out >= 0) p->dt_out = dt_out;
    p->r0 = 0; p->r1 = n;
    const int e = run_forward(p, q, k, v, h, shared, y, st, &launches);
    p->r0 = 0; p->r1 = (long long)p->B * p->C;
    p->h_dtype = p->dtype;
    p->dt_in = p->dt_out = p->dt_in2 = p->dt_out2 = p->dtype;
    return e;
}

// y = q (h conv (k v)) and y2 = q2 (h' conv (k2 v2)), h'[d] = h[-d], in one pass over the groups of the plan (multi-kernel
// paths): the spectrum of h' is the conjugate of the spectrum of h under the wrapped tap placement (real taps), so the
// second signal side reuses the filter spectrum its group has just computed.  In causal mode h' is the anti-causal
// kernel: supports [0, L) and [-(L-1), 0] on a ring of P >= 2L-1 points still do not wrap into the kept outputs.
static int grad_forward_pair(hyenand_plan *p, long long n, const void *q, const void *k, const void *v, void *y,
                             const void *q2, const void *k2, const void *v2, void *y2, const void *h, bool shared,
                             cudaStream_t st, int h_dtype, int dt_in = HYENAND_F32, int dt_out = HYENAND_F32,
                             int dt_in2 = HYENAND_F32, int dt_out2 = HYENAND_F32)
{
    p->q2 = (const char *)q2; p->k2 = (const char *)k2; p->v2 = (const char *)v2; p->y2 = (char *)y2;
    p->dt_in = dt_in; p->dt_out = dt_out; p->dt_in2 = dt_in2; p->dt_out2 = dt_out2;
    const int e = grad_forward(p, n, (const float *)q, (const float *)k, (const float *)v, h, shared, (float *)y, st, h_dtype);
    p->q2 = p->k2 = p->v2 = nullptr; p->y2 = nullptr;
    return e;
}

extern "C" int hyenand_backward(hyenand_grad *g, const void *q, const void *k, const void *v, const void *h,
                                long long h_batch_stride_elems, const void *dy, void *dq, void *dk, void *dv, void *dh,
                                void *cuda_stream)
{
    g_err[0] = 0;
    if (!g) return fail(HYENAND_ERR_INVALID_ARG, "handle is NULL");
    const void *ptrs[9] = {q, k, v, h, dy, dq, dk, dv, dh};
    for (int i = 0; i < 9; ++i) {
        if (!ptrs[i]) return fail(HYENAND_ERR_INVALID_ARG, "pointer %d is NULL", i);
        if (((uintptr_t)ptrs[i]) & 15) return fail(HYENAND_ERR_INVALID_ARG, "pointer %d is not 16-byte aligned", i);
    }
    bool shared = false;
    if (h_batch_stride_elems == 0) shared = true;
    else if (h_batch_stride_elems != (long long)g->C * g->kvol)
        return fail(HYENAND_ERR_INVALID_ARG, "h_batch_stride_elems must be 0 or C*K_1*..*K_N = %lld", (long long)g->C * g->kvol);
    int e = check_device(g->main);
    if (e) return e;
    {
        // no output may overlap an input or another output: the kernels write the gradients while they read the inputs
        const size_t nb_ = (size_t)g->B * g->C * g->vol * elsize(g->dtype);
        const size_t hb_ = (size_t)(shared ? 1 : g->B) * g->C * g->kvol * elsize(g->dtype);
        const size_t len[9] = {nb_, nb_, nb_, hb_, nb_, nb_, nb_, nb_, hb_};
        for (int o = 5; o < 9; ++o)
            for (int i = 0; i < o; ++i) {
                const char *a = (const char *)ptrs[o], *b = (const char *)ptrs[i];
                if (a < b + len[i] && b < a + len[o])
                    return fail(HYENAND_ERR_INVALID_ARG, "output %d overlaps pointer %d", o, i);
            }
    }
    {
        DbgScope d;
        const size_t nbytes = (size_t)g->B * g->C * g->vol * elsize(g->dtype);
        const size_t hbytes = (size_t)(shared ? 1 : g->B) * g->C * g->kvol * elsize(g->dtype);
        d.add(q, nbytes); d.add(k, nbytes); d.add(v, nbytes); d.add(dy, nbytes); d.add(dq, nbytes); d.add(dk, nbytes); d.add(dv, nbytes);
        d.add(h, hbytes); d.add(dh, hbytes);
        d.add(g->allocs); d.add(g->main->allocs);
        if (g->adj != g->main) d.add(g->adj->allocs);
        if (g->caus && g->caus != g->main) d.add(g->caus->allocs);
        d.commit();
    }
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const size_t es = elsize(g->dtype);
    const bool widen = g->dtype == HYENAND_BF16;
    const long long C = g->C, vol = g->vol, kvol = g->kvol;
    const int *L = g->L, *K = g->K;
    const bool nat = widen && g->h_native;                     // bf16 taps go to the transforms as they are
    const int hdt = nat ? HYENAND_BF16 : HYENAND_F32;
    const float *hsh = (const float *)h;                       // shared kernel, fp32 view
    if (shared && widen && !nat) { launch_widen(h, g->dtype, C * kvol, g->h32, st); hsh = g->h32; }
    for (int b0 = 0; b0 < g->B; b0 += g->nb) {
        const long long n = g->B - b0 < g->nb ? g->B - b0 : g->nb, S = n * C, off = (long long)b0 * C * vol;
        const float *q32 = (const float *)q + off, *k32 = (const float *)k + off, *v32 = (const float *)v + off, *dy32 = (const float *)dy + off;
        if (widen && !g->native) {
            launch_widen((const char *)q + off * es, g->dtype, S * vol, g->q32, st); q32 = g->q32;
            launch_widen((const char *)k + off * es, g->dtype, S * vol, g->k32, st); k32 = g->k32;
            launch_widen((const char *)v + off * es, g->dtype, S * vol, g->v32, st); v32 = g->v32;
            launch_widen((const char *)dy + off * es, g->dtype, S * vol, g->dy32, st); dy32 = g->dy32;
        }
        const float *h32 = hsh;                                  // (bf16 taps when nat)
        if (!shared) {
            h32 = (const float *)((const char *)h + (long long)b0 * C * kvol * es);
            if (widen && !nat) { launch_widen((const char *)h + (long long)b0 * C * kvol * es, g->dtype, S * kvol, g->h32, st); h32 = g->h32; }
        }
        const long long Sh = shared ? C : S;
        // the caller's tensors of this pass, in their own element type
        const char *qn = (const char *)q + off * es, *kn = (const char *)k + off * es, *vn = (const char *)v + off * es,
                   *dyn = (const char *)dy + off * es;
        if (g->two_gate) {
            // the plan runs in the caller's element type: dq = dy * (h conv (k v)) is a forward gated by dy; the forward of
            // dy q against the kernel at the opposite displacement leaves through two gates, dk = v * du and dv = k * du
            char *dqn = (char *)dq + off * es, *dkn = (char *)dk + off * es, *dvn = (char *)dv + off * es;
            if ((e = grad_forward(g->main, S, (const float *)dyn, (const float *)kn, (const float *)vn, h32, shared, (float *)dqn, st, g->dtype)))
                return e;
            RemapArgs r{};
            r.a = h32; r.b = nullptr; r.out = g->hopp; r.slices = Sh;
            r.a_bf16 = r.out_bf16 = widen;
            for (int a = 0; a < 3; ++a) { r.Ls[a] = K[a]; r.G[a] = K[a]; r.mode[a] = REMAP_REV; }
            launch_remap(r, st);
            g->main->qg2 = kn; g->main->yg2 = dvn;
            e = grad_forward(g->main, S, (const float *)vn, (const float *)dyn, (const float *)qn, g->hopp, shared, (float *)dkn, st, g->dtype);
            g->main->qg2 = nullptr; g->main->yg2 = nullptr;
            if (e) return e;
        } else if (g->native && g->pair) {
            // as below, on the caller's bf16 tensors: the first side is a bf16 forward with dy as its gate and dq as its
            // result, the second reads dy and q and leaves through two gates, dk = v * du and dv = k * du
            g->main->qg2 = kn; g->main->yg2 = (char *)dv + off * es;
            e = grad_forward_pair(g->main, S, dyn, kn, vn, (char *)dq + off * es, vn, dyn, qn, (char *)dk + off * es, h32, shared, st, hdt,
                                  HYENAND_BF16, HYENAND_BF16, HYENAND_BF16, HYENAND_BF16);
            g->main->qg2 = nullptr; g->main->yg2 = nullptr;
            if (e) return e;
        } else if (g->pair) {
            // dq = dy * (h conv (k v)) and du = h' conv (dy q) from one pass over the groups; dk = du v, dv = du k
            if (!widen) {
                // fp32 I/O: every gradient is written in place, the second side leaves through two gates (dk = v du, dv = k du)
                g->main->qg2 = (const char *)k32; g->main->yg2 = (char *)((float *)dv + off);
                e = grad_forward_pair(g->main, S, dy32, k32, v32, (float *)dq + off, v32, dy32, q32, (float *)dk + off, h32, shared, st, hdt);
                g->main->qg2 = nullptr; g->main->yg2 = nullptr;
                if (e) return e;
            } else {
                if ((e = grad_forward_pair(g->main, S, dy32, k32, v32, g->t32, nullptr, dy32, q32, g->aux, h32, shared, st, hdt))) return e;
                launch_mul_cast(g->t32, nullptr, 0, S * vol, g->dtype, (char *)dq + off * es, st);
                launch_mul_cast(g->aux, v32, 0, S * vol, g->dtype, (char *)dk + off * es, st);
                launch_mul_cast(g->aux, k32, 0, S * vol, g->dtype, (char *)dv + off * es, st);
            }
        } else if (g->long1d && g->mode == HYENAND_MODE_CAUSAL) {
            // dq = dy * (h conv (k v)); with ct_native a forward on the caller's bf16 tensors, dq written in place
            const bool cn = g->ct_native;
            if (cn) {
                if ((e = grad_forward(g->main, S, (const float *)dyn, (const float *)kn, (const float *)vn, h32, shared,
                                      (float *)((char *)dq + off * es), st, hdt, g->dtype, g->dtype))) return e;
            } else {
                if ((e = grad_forward(g->main, S, dy32, k32, v32, h32, shared, g->t32, st, hdt))) return e;
                launch_mul_cast(g->t32, nullptr, 0, S * vol, g->dtype, (char *)dq + off * es, st);
            }
            // du[t] = sum_{s >= t} h[s - t] g[s], g = dy q, is the anti-causal convolution; read backwards in time it is
            // the causal one, rev(du) = h conv rev(g): the causal plan (and its faster kernels) serves, with two
            // reversals at the copy rate, instead of a non-causal plan with a kernel of 2L-1 taps, half of them zero.
            // aux = rev(g) stays for the dh stage below.
            RemapArgs r{};
            r.a = dy32; r.b = q32; r.out = g->aux; r.slices = S;
            if (cn) { r.a = (const float *)dyn; r.b = (const float *)qn; r.a_bf16 = 1; }
            for (int a = 0; a < 3; ++a) { r.Ls[a] = L[a]; r.G[a] = L[a]; r.mode[a] = a == 2 ? REMAP_REV : REMAP_PAD; }
            launch_remap(r, st);
            g->main->ct.keep_filter = shared;                       // same taps as the forward for dq just before
            e = grad_forward(g->main, S, g->ones, g->aux, g->ones, h32, shared, g->t32, st, hdt, HYENAND_F32, HYENAND_F32);
            g->main->ct.keep_filter = 0;
            if (e) return e;
            RemapArgs rv{};
            rv.a = g->t32; rv.out = g->hopp; rv.slices = S;          // hopp: S*(2L-1) floats, du takes the first S*L
            for (int a = 0; a < 3; ++a) { rv.Ls[a] = L[a]; rv.G[a] = L[a]; rv.mode[a] = a == 2 ? REMAP_REV : REMAP_PAD; }
            launch_remap(rv, st);
            launch_mul_cast(g->hopp, cn ? (const void *)vn : (const void *)v32, cn ? g->dtype : 0, S * vol, g->dtype, (char *)dk + off * es, st);
            launch_mul_cast(g->hopp, cn ? (const void *)kn : (const void *)k32, cn ? g->dtype : 0, S * vol, g->dtype, (char *)dv + off * es, st);
        } else {
            // dq = dy * (h conv (k v))
            if ((e = grad_forward(g->main, S, dy32, k32, v32, h32, shared, g->t32, st, hdt))) return e;
            launch_mul_cast(g->t32, nullptr, 0, S * vol, g->dtype, (char *)dq + off * es, st);
            // the kernel at the opposite displacement
            {
                RemapArgs r{};
                r.a = h32; r.b = nullptr; r.out = g->hopp; r.slices = Sh;
                r.a_bf16 = r.out_bf16 = nat;
                for (int a = 0; a < 3; ++a) {
                    r.Ls[a] = K[a]; r.G[a] = K[a];
                    r.mode[a] = g->mode == HYENAND_MODE_CIRCULAR ? REMAP_NEG : REMAP_REV;
                }
                if (g->mode == HYENAND_MODE_CAUSAL) r.G[2] = 2 * L[2] - 1;       // causal taps as the negative half of a non-causal kernel
                launch_remap(r, st);
            }
            // du = h' conv (dy q);  dk = du v, dv = du k
            if ((e = grad_forward(g->adj, S, g->ones, dy32, q32, g->hopp, shared, g->t32, st, hdt))) return e;
            launch_mul_cast(g->t32, v32, 0, S * vol, g->dtype, (char *)dk + off * es, st);
            launch_mul_cast(g->t32, k32, 0, S * vol, g->dtype, (char *)dv + off * es, st);
        }
        // dh
        float *dhS = shared ? g->dhs : g->dh32;                  // per-slice kernel gradients of this pass
        bool dh_direct = false;                                  // this pass's dh is already in the caller's tensor
        if (g->mode == HYENAND_MODE_CIRCULAR) {
            // dh[m] = sum_i g_i u_{(i-m) mod L}: circular convolution of g with u read at the opposite displacement
            // (hopp is free again: the forward that consumed the opposite kernel precedes this on the stream)
            RemapArgs r{};
            r.a = k32; r.b = v32; r.out = g->hopp; r.slices = S;
            for (int a = 0; a < 3; ++a) { r.Ls[a] = L[a]; r.G[a] = L[a]; r.mode[a] = REMAP_NEG; }
            launch_remap(r, st);
            if ((e = grad_forward(g->main, S, g->ones, dy32, q32, g->hopp, false, dhS, st))) return e;
            if (shared) launch_batch_sum(dhS, n, C, kvol, b0 == 0, g->dh32, st);
        } else if (g->long1d) {
            const int Ln = L[2];
            // Displacements d >= 0: dh[d] = sum_s g_{s+d} u_s.  The causal forward with the reversed g as its kernel gives
            // c[n] = sum_{s<=n} g[L-1-(n-s)] u_s, and c[L-1-d] is that sum.
            RemapArgs r{};
            r.a = dy32; r.b = q32; r.out = g->aux; r.slices = S;
            for (int a = 0; a < 3; ++a) { r.Ls[a] = L[a]; r.G[a] = L[a]; r.mode[a] = a == 2 ? REMAP_REV : REMAP_PAD; }
            if (g->mode != HYENAND_MODE_CAUSAL) launch_remap(r, st);       // (causal: aux holds the reversed g already)
            if (g->ct_native)       // k and v as they are, the kernel (reversed g) and the result in fp32
                e = grad_forward(g->caus, S, g->ones, (const float *)kn, (const float *)vn, g->aux, false, g->t32, st, HYENAND_F32,
                                 g->dtype, HYENAND_F32);
            else
                e = grad_forward(g->caus, S, g->ones, k32, v32, g->aux, false, g->t32, st);
            if (e) return e;
            if (g->mode == HYENAND_MODE_CAUSAL) {
                RemapArgs w{};                                 // tap t <- c[L-1-t]
                w.a = g->t32; w.out = dhS; w.slices = S;
                for (int a = 0; a < 3; ++a) { w.Ls[a] = L[a]; w.G[a] = K[a]; w.mode[a] = a == 2 ? REMAP_REV : REMAP_PAD; }
                launch_remap(w, st);
            } else {
                // Displacements -t < 0: dh[-t] = sum_s u_{s+t} g_s, the same form with g and u exchanged: c'[L-1-t].
                // Tap m = d + L-1: the lower taps m = 0..L-1 are c'[m] (a plain copy), the upper taps m = L..2L-2 are
                // c[2(L-1)-m], the reversed c from its second entry on.
                r.a = k32; r.b = v32;
                launch_remap(r, st);                           // reversed u (the forward that read aux precedes this on the stream)
                float *neg = g->hopp;                          // S*(2L-1) floats, free again
                if ((e = grad_forward(g->caus, S, g->ones, dy32, q32, g->aux, false, neg, st))) return e;
                RemapArgs lo{};
                lo.a = neg; lo.out = dhS; lo.slices = S;
                for (int a = 0; a < 3; ++a) { lo.Ls[a] = L[a]; lo.G[a] = K[a]; lo.mode[a] = REMAP_PAD; }
                launch_remap(lo, st);
                RemapArgs rv{};
                rv.a = g->t32; rv.out = g->aux; rv.slices = S;
                for (int a = 0; a < 3; ++a) { rv.Ls[a] = L[a]; rv.G[a] = L[a]; rv.mode[a] = a == 2 ? REMAP_REV : REMAP_PAD; }
                launch_remap(rv, st);                          // aux[j] = c[L-1-j] = dh[d = j]
                if (Ln > 1 &&
                    cudaMemcpy2DAsync(dhS + Ln, (size_t)kvol * sizeof(float), g->aux + 1, (size_t)vol * sizeof(float),
                                      (size_t)(Ln - 1) * sizeof(float), (size_t)S, cudaMemcpyDeviceToDevice, st) != cudaSuccess)
                    return fail(HYENAND_ERR_CUDA, "copy of the upper taps failed: %s", cudaGetErrorString(cudaGetLastError()));
            }
            if (shared) launch_batch_sum(dhS, n, C, kvol, b0 == 0, g->dh32, st);
        } else {
            // dh[m] = sum_t g_t u_{t - d}, m = d + L-1: the full linear convolution of g = dy q with the reversed u = k v,
            // ns slices at a time
            {
                RemapArgs r{};
                r.a = k32; r.b = v32; r.out = g->aux; r.slices = S;
                if (g->native) { r.a = (const float *)kn; r.b = (const float *)vn; r.a_bf16 = 1; }
                for (int a = 0; a < 3; ++a) { r.Ls[a] = L[a]; r.G[a] = L[a]; r.mode[a] = REMAP_REV; }
                launch_remap(r, st);
            }
            // Per-sample kernels without a causal crop: the last stage writes the caller's dh itself (one rounding of the
            // fp32 sums either way), else fp32 taps that are cropped and/or summed over the batch below.
            dh_direct = !shared && g->mode != HYENAND_MODE_CAUSAL;
            char *dh_pass = (char *)dh + (long long)b0 * C * kvol * es;
            float *full = g->mode == HYENAND_MODE_CAUSAL ? g->hopp : dhS;     // all 2L-1 taps per slice
            for (long long s0 = 0; s0 < S; s0 += g->ns) {
                const long long m = S - s0 < g->ns ? S - s0 : g->ns;
                void *dst = dh_direct ? (void *)(dh_pass + s0 * kvol * es) : (void *)(full + s0 * g->kopp);
                const void *gy = g->native ? (const void *)(dyn + s0 * vol * es) : (const void *)(dy32 + s0 * vol);
                const void *gq = g->native ? (const void *)(qn + s0 * vol * es) : (const void *)(q32 + s0 * vol);
                if ((e = corr_dh(g, m, gy, gq, g->native ? g->dtype : HYENAND_F32, g->aux + s0 * vol, dst,
                                 dh_direct ? g->dtype : HYENAND_F32, st)))
                    return e;
            }
            if (g->mode == HYENAND_MODE_CAUSAL &&
                cudaMemcpy2DAsync(dhS, (size_t)kvol * sizeof(float), g->hopp + (L[2] - 1), (size_t)g->kopp * sizeof(float),
                                  (size_t)kvol * sizeof(float), (size_t)S, cudaMemcpyDeviceToDevice, st) != cudaSuccess)
                return fail(HYENAND_ERR_CUDA, "copy of the causal taps failed: %s", cudaGetErrorString(cudaGetLastError()));
            if (shared) launch_batch_sum(dhS, n, C, kvol, b0 == 0, g->dh32, st);
        }
        if (!shared && !dh_direct) launch_mul_cast(g->dh32, nullptr, 0, S * kvol, g->dtype, (char *)dh + (long long)b0 * C * kvol * es, st);
    }
    if (shared) launch_mul_cast(g->dh32, nullptr, 0, C * kvol, g->dtype, dh, st);
    cudaError_t ce = cudaGetLastError();
    if (ce != cudaSuccess) return fail(HYENAND_ERR_CUDA, "kernel launch failed: %s", cudaGetErrorString(ce));
    return HYENAND_OK;
}

extern "C" long long hyenand_backward_guard_damage(hyenand_grad *g)
{
    g_err[0] = 0;
    if (!g) { fail(HYENAND_ERR_INVALID_ARG, "handle is NULL"); return -1; }
    long long bad = guard_damage(&g->allocs);
    hyenand_plan *plans[4] = {g->main, g->adj != g->main ? g->adj : nullptr, nullptr, (g->caus && g->caus != g->main) ? g->caus : nullptr};
    for (int i = 0; i < 4 && bad >= 0; ++i)
        if (plans[i]) { const long long b = guard_damage(&plans[i]->allocs); bad = b < 0 ? -1 : bad + b; }
    return bad;
}

// ---- kernel synthesis ---------------------------------------------------------------------------------

extern "C" int hyenand_synth_device_status(void) { return synth_device_status(); }


extern "C" int hyenand_synthesize_kernel(int ndim, const int *dims, int mode, int B, int C, int hidden, int layers,
                                         const float *W1, const float *b1, const float *omega0, const float *Wh,
                                         const float *bh, const float *Wout, const float *bout, const float *gamma,
                                         const float *beta, const float *window, int dtype, void *h, void *cuda_stream)
{
    g_err[0] = 0;
    if (ndim < 1 || ndim > 3 || !dims) return fail(HYENAND_ERR_INVALID_ARG, "ndim must be 1, 2 or 3 and dims non-NULL");
    if (mode != HYENAND_MODE_LINEAR && mode != HYENAND_MODE_CAUSAL && mode != HYENAND_MODE_CIRCULAR)
        return fail(HYENAND_ERR_INVALID_ARG, "unknown boundary mode %d", mode);
    if (mode == HYENAND_MODE_CAUSAL && ndim != 1) return fail(HYENAND_ERR_UNSUPPORTED, "causal kernels are defined for 1-D grids only");
    if (B < 1 || C < 1) return fail(HYENAND_ERR_INVALID_ARG, "B and C must be >= 1");
    if (dtype != HYENAND_F32 && dtype != HYENAND_BF16) return fail(HYENAND_ERR_INVALID_ARG, "unknown dtype %d", dtype);
    if (!synth_supported(hidden, layers))
        return fail(HYENAND_ERR_UNSUPPORTED, "hidden width must be 1..64 and the number of hidden layers 1..8 (got %d, %d)", hidden, layers);
    if (!W1 || !b1 || !omega0 || !Wout || !bout || !window || !h || (layers > 1 && (!Wh || !bh)))
        return fail(HYENAND_ERR_INVALID_ARG, "a parameter pointer is NULL");
    if ((gamma == nullptr) != (beta == nullptr)) return fail(HYENAND_ERR_INVALID_ARG, "gamma and beta are given together or not at all");
    if (((uintptr_t)h) & 15) return fail(HYENAND_ERR_INVALID_ARG, "h is not 16-byte aligned");
    SynthArgs a{};
    a.ndim = ndim; a.mode = mode; a.B = B; a.C = C; a.hidden = hidden; a.layers = layers;
    for (int x = 0; x < 3; ++x) { a.L[x] = 1; a.K[x] = 1; }
    for (int x = 0; x < ndim; ++x) {
        if (dims[x] < 1) return fail(HYENAND_ERR_INVALID_ARG, "dims[%d] = %d must be >= 1", x, dims[x]);
        a.L[3 - ndim + x] = dims[x];
        a.K[3 - ndim + x] = mode == HYENAND_MODE_LINEAR ? 2 * dims[x] - 1 : dims[x];
    }
    a.W1 = W1; a.b1 = b1; a.omega0 = omega0; a.Wh = Wh; a.bh = bh; a.Wout = Wout; a.bout = bout;
    a.gamma = gamma; a.beta = beta; a.window = window; a.h = h; a.dtype = dtype;
    static const bool alu_only = getenv("HYENAND_SYNTH_ALU") != nullptr;     // development switch, read once
    a.no_tensor_cores = alu_only;
    {
        DbgScope d;
        const size_t f = sizeof(float);
        d.add(W1, f * hidden * ndim); d.add(b1, f * hidden); d.add(omega0, f * hidden);
        d.add(Wh, f * (size_t)(layers - 1) * hidden * hidden); d.add(bh, f * (size_t)(layers - 1) * hidden);
        d.add(Wout, f * (size_t)C * hidden); d.add(bout, f * C);
        d.add(gamma, f * (size_t)B * layers * hidden); d.add(beta, f * (size_t)B * layers * hidden);
        d.add(window, f * (size_t)(mode == HYENAND_MODE_CAUSAL ? C : ndim * C));
        d.add(h, (size_t)B * C * a.K[0] * a.K[1] * a.K[2] * elsize(dtype));
        d.commit();
    }
    if (launch_synth(a, (cudaStream_t)cuda_stream) < 0) return fail(HYENAND_ERR_UNSUPPORTED, "kernel grid too large for one launch");
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return fail(HYENAND_ERR_CUDA, "kernel launch failed: %s", cudaGetErrorString(e));
    return HYENAND_OK;
}

// ---- forward without any device allocation --------------------------------------------------
//
// Some callers may not allocate device memory at the point where they need the operator: code
// running while a CUDA graph is being captured elsewhere in the process, inside a memory pool's
// critical section, or in a service whose device memory was fully handed out at start-up.  For
// them the workspace of this entry point is a fixed array inside the library image.

#define HYENAND_NOALLOC_MAX_BYTES (16u << 20)

static __device__ __align__(256) unsigned char g_noalloc_scratch[HYENAND_NOALLOC_MAX_BYTES];

// device address of g_noalloc_scratch per device ordinal, resolved on that device's first call
static void *g_noalloc_ptr[64] = {nullptr};

__global__ void noalloc_twiddle_kernel(float2 *tw, int n)
{
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t < n) {
        double sn, cs;
        sincospi(-2.0 * (double)t / (double)n, &sn, &cs);
        tw[t] = make_float2((float)cs, (float)sn);
    }
}

extern "C" size_t hyenand_noalloc_max_bytes(void) { return HYENAND_NOALLOC_MAX_BYTES; }

extern "C" int hyenand_forward_noalloc(int ndim, const int *dims, int B, int C, int causal, int dtype,
                                       const void *q, const void *k, const void *v, const void *h,
                                       long long h_batch_stride_elems, void *y, void *cuda_stream)
{
    g_err[0] = 0;
    if (ndim < 1 || ndim > 3 || !dims) return fail(HYENAND_ERR_INVALID_ARG, "ndim must be 1, 2 or 3 and dims non-NULL");
    if (B < 1 || C < 1) return fail(HYENAND_ERR_INVALID_ARG, "B and C must be >= 1");
    if (dtype != HYENAND_F32 && dtype != HYENAND_BF16) return fail(HYENAND_ERR_INVALID_ARG, "unknown dtype %d", dtype);
    if (causal != 0 && causal != 1) return fail(HYENAND_ERR_INVALID_ARG, "causal must be 0 or 1");
    if (causal && ndim != 1) return fail(HYENAND_ERR_UNSUPPORTED, "causal kernels are defined for 1-D grids only");
    if (!q || !k || !v || !h || !y) return fail(HYENAND_ERR_INVALID_ARG, "q, k, v, h, y must be non-NULL");
    const void *ptrs[5] = {q, k, v, h, y};
    for (int i = 0; i < 5; ++i)
        if (((uintptr_t)ptrs[i]) & 15) return fail(HYENAND_ERR_INVALID_ARG, "pointer %d is not 16-byte aligned", i);

    // geometry of a throw-away plan that lives on this call's stack (no host or device allocation)
    static thread_local hyenand_plan sp;
    memset(&sp, 0, sizeof(sp));
    hyenand_plan *p = &sp;
    p->ndim = ndim; p->B = B; p->C = C; p->causal = causal; p->dtype = dtype; p->h_dtype = dtype;
    p->dt_in = p->dt_out = p->dt_in2 = p->dt_out2 = dtype;
    p->r0 = 0; p->r1 = (long long)B * C;
    p->vol = 1; p->kvol = 1;
    for (int a = 0; a < 3; ++a) { p->L[a] = 1; p->K[a] = 1; p->P[a] = 1; p->log2p[a] = 0; }
    for (int a = 0; a < ndim; ++a) {
        const int ia = 3 - ndim + a;
        if (dims[a] < 1) return fail(HYENAND_ERR_INVALID_ARG, "dims[%d] = %d must be >= 1", a, dims[a]);
        if (dims[a] > (1 << (kMaxLineLog2 - 1)))
            return fail(HYENAND_ERR_UNSUPPORTED, "dims[%d] = %d exceeds the limit of %d of the allocation-free entry point",
                        a, dims[a], 1 << (kMaxLineLog2 - 1));
        p->dims[a] = dims[a];
        p->L[ia] = dims[a];
        p->K[ia] = causal ? dims[a] : 2 * dims[a] - 1;
        p->log2p[ia] = next_pow2_log(2 * dims[a] - 1);
        p->P[ia] = 1 << p->log2p[ia];
        p->vol *= dims[a];
        p->kvol *= p->K[ia];
    }
    p->XH = p->P[2] / 2 + 1;
    p->XP = (p->XH + 1) & ~1;
    p->path = PATH_ND_GENERIC;
    bool shared = false;
    int e = check_stride(p, h_batch_stride_elems, &shared);
    if (!e) e = check_overlap(p, shared, q, k, v, h, y);
    if (e) return e;
    const bool three = p->P[0] > 1;
    p->ws_a_slice = (long long)p->L[0] * p->L[1] * p->XP;
    p->wh_a_slice = (long long)p->K[0] * p->K[1] * p->XP;
    p->ws_b_slice = three ? (long long)p->L[0] * p->P[1] * p->XP : 0;
    p->wh_b_slice = three ? (long long)p->K[0] * p->P[1] * p->XP : 0;
    int gl = 1;
    for (int a = 0; a < 3; ++a) if (p->log2p[a] > gl) gl = p->log2p[a];
    p->gtw_n = 1 << gl;

    // carve the fixed array: twiddles, then k*v spectra, then filter spectra (256-byte granules)
    auto up = [](unsigned long long x) { return (x + 255ull) & ~255ull; };
    const unsigned long long S = (unsigned long long)B * C;
    const unsigned long long tw_b = up(sizeof(float2) * (unsigned long long)p->gtw_n);
    const unsigned long long ua = up(sizeof(float2) * (unsigned long long)p->ws_a_slice), ub = up(sizeof(float2) * (unsigned long long)p->ws_b_slice);
    const unsigned long long ha = up(sizeof(float2) * (unsigned long long)p->wh_a_slice), hb2 = up(sizeof(float2) * (unsigned long long)p->wh_b_slice);
    const unsigned long long fixed = tw_b + (shared ? (unsigned long long)C * (ha + hb2) : 0ull);
    const unsigned long long per = ua + ub + (shared ? 0ull : ha + hb2);
    if (fixed + per > HYENAND_NOALLOC_MAX_BYTES)
        return fail(HYENAND_ERR_UNSUPPORTED,
                    "problem needs %llu bytes of workspace for one slice%s; the allocation-free entry point has %u bytes",
                    fixed + per, shared ? " plus the shared filters" : "", HYENAND_NOALLOC_MAX_BYTES);
    unsigned long long spc = (HYENAND_NOALLOC_MAX_BYTES - fixed) / per;
    if (spc > S) spc = S;
    p->slices_per_chunk = (long long)spc;
    p->n_lanes = 1;
    hyenand_plan::Lane &ln = p->lane[0];
    ln.wh_slices = shared ? C : (long long)spc;

    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64)
        return fail(HYENAND_ERR_CUDA, "cannot identify the current device");
    p->device = dev;
    if (!g_noalloc_ptr[dev]) {
        // once per device, with that device current: the array's name is only a host-side handle
        void *ptr = nullptr;
        cudaError_t ce = cudaGetSymbolAddress(&ptr, g_noalloc_scratch);
        if (ce != cudaSuccess || !ptr)
            return fail(HYENAND_ERR_CUDA, "cudaGetSymbolAddress failed: %s", cudaGetErrorString(ce));
        g_noalloc_ptr[dev] = ptr;
    }
    unsigned char *base = (unsigned char *)g_noalloc_ptr[dev];
    unsigned long long off = 0;
    p->gtw = (float2 *)(base + off); off += tw_b;
    ln.ws_a = (float2 *)(base + off); off += ua * spc;
    ln.ws_b = three ? (float2 *)(base + off) : nullptr; off += ub * spc;
    ln.wh_a = (float2 *)(base + off); off += ha * (unsigned long long)ln.wh_slices;
    ln.wh_b = three ? (float2 *)(base + off) : nullptr; off += hb2 * (unsigned long long)ln.wh_slices;
    // the per-slice strides used by the kernels are the unrounded ones; the carve only has to be large enough
    {
        DbgScope d;
        const size_t nbytes = (size_t)B * C * p->vol * elsize(dtype);
        d.add(q, nbytes); d.add(k, nbytes); d.add(v, nbytes); d.add(y, nbytes);
        d.add(h, (size_t)(shared ? 1 : B) * C * p->kvol * elsize(dtype));
        d.add(base, HYENAND_NOALLOC_MAX_BYTES);
        d.commit();
    }
    cudaStream_t st = (cudaStream_t)cuda_stream;
    noalloc_twiddle_kernel<<<(p->gtw_n + 255) / 256, 256, 0, st>>>(p->gtw, p->gtw_n);
    int launches = 1;
    return run_forward(p, q, k, v, h, shared, y, st, &launches);
}
