// Shared declarations of the library's translation units (internal).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace hn {

typedef __nv_bfloat16 bf16;

// ---- checked build -----------------------------------------------------------------------------------------
// With -DHYENAND_DEBUG (libhyenand_debug.so) every access to global memory that a kernel makes through its own
// instructions (loads, stores, asynchronous copies, L2 prefetches; tensor copies are bounded by their tensor maps) is
// first compared with the list of address ranges the call may touch: the caller's tensors and the device allocations
// of the objects involved.  An access outside all of them is counted, with its address and source line; the access
// itself is still made (the checked build must behave like the product build).  It stands in for a memory checker
// on machines where none can be run.  Each translation unit holds its own copy of the list and of the counters
// (no relocatable device code), kept in step by hooks registered at load time.
constexpr int kDbgRanges = 96;
struct DbgRanges {
    unsigned long long lo[kDbgRanges], hi[kDbgRanges];
    int n;
};
struct DbgReport {
    unsigned long long count, first_address;
    int first_line;
    const char *file;
};
typedef void (*DbgHook)(const DbgRanges *set, unsigned long long *collect);
void dbg_register(DbgHook hook, const char *file);
void dbg_set_ranges(const DbgRanges &r);
void dbg_append_range(const void *ptr, size_t bytes);     // one more range for the call in progress           // uploads to every translation unit
DbgReport dbg_collect();                           // sums and clears the counters of every translation unit
}  // namespace hn

#ifdef HYENAND_DEBUG
static __device__ hn::DbgRanges hn_dbg_ranges;
static __device__ unsigned long long hn_dbg_bad[4];        // count, first address, first line
namespace hn {
__device__ __forceinline__ void dbg_check(const void *p, unsigned bytes, int line)
{
    if (!__isGlobal(p)) return;                            // generic pointers into shared memory are not this check's business
    const unsigned long long a = (unsigned long long)p;
    bool ok = false;
    for (int i = 0; i < hn_dbg_ranges.n; ++i) ok |= a >= hn_dbg_ranges.lo[i] && a + bytes <= hn_dbg_ranges.hi[i];
    if (!ok && atomicAdd(&hn_dbg_bad[0], 1ull) == 0) { hn_dbg_bad[1] = a; hn_dbg_bad[2] = (unsigned long long)line; }
}
}  // namespace hn
static void hn_dbg_hook(const hn::DbgRanges *set, unsigned long long *collect)
{
    if (set) cudaMemcpyToSymbol(hn_dbg_ranges, set, sizeof(*set));
    if (collect) {
        cudaMemcpyFromSymbol(collect, hn_dbg_bad, sizeof(unsigned long long) * 4);
        const unsigned long long zero[4] = {0, 0, 0, 0};
        cudaMemcpyToSymbol(hn_dbg_bad, zero, sizeof(zero));
    }
}
namespace { struct HnDbgRegistrar { HnDbgRegistrar() { hn::dbg_register(hn_dbg_hook, __BASE_FILE__); } } hn_dbg_registrar; }
#define HN_G(p, bytes) hn::dbg_check((p), (unsigned)(bytes), __LINE__)
#else
#define HN_G(p, bytes) ((void)0)
#endif

namespace hn {

template <typename T> struct IO;
template <> struct IO<float> {
    static __device__ __forceinline__ float ld(const float *p, long long i) { HN_G(p + i, 4); return __ldg(p + i); }
    static __device__ __forceinline__ void st(float *p, long long i, float v) { HN_G(p + i, 4); p[i] = v; }
};
template <> struct IO<bf16> {
    static __device__ __forceinline__ float ld(const bf16 *p, long long i)
    {
        HN_G(p + i, 2);
        return __bfloat162float(__ldg(p + i));
    }
    static __device__ __forceinline__ void st(bf16 *p, long long i, float v) { HN_G(p + i, 2); p[i] = __float2bfloat16_rn(v); }
};

// Optional per-kernel timing: when enabled, every kernel launch of a forward is
// bracketed by CUDA events on the launching stream; collect() (after the caller
// synchronised) adds the elapsed times to per-kernel totals.
enum KernelId {
    KID_ROWS_H = 0, KID_AXIS_H, KID_ROWS_U, KID_AXIS_U, KID_CORE, KID_AXIS_INV, KID_ROWS_INV,
    KID_CT_COLS_H, KID_CT_COLS_U, KID_CT_CORE, KID_CT_COLS_INV, KID_PLANE_H, KID_PLANE_U, KID_PLANE_INV, KID_FUSED2D, KID_CT_HSPEC, KID_COUNT
};

// names of the KernelId entries (hyenand.cu)
extern const char *const kKernelNames[];
// NVTX range around a launch (a no-op unless a profiler that consumes NVTX is attached)
void nvtx_push(const char *name);
void nvtx_pop();

struct Prof {
    bool on = false;
    bool nvtx = false;                // HYENAND_NVTX at plan creation: one NVTX range per kernel launch
    struct Rec { cudaEvent_t a, b; int kid; };
    Rec recs[4096];
    int created = 0, used = 0;
    double ms[KID_COUNT] = {0};
    long long launches[KID_COUNT] = {0};
    void begin(int kid, cudaStream_t st)
    {
        if (nvtx) nvtx_push(kKernelNames[kid]);
        if (!on || used >= 4096) return;
        if (used == created) {
            cudaEventCreate(&recs[created].a);
            cudaEventCreate(&recs[created].b);
            ++created;
        }
        recs[used].kid = kid;
        cudaEventRecord(recs[used].a, st);
    }
    void end(cudaStream_t st)
    {
        if (nvtx) nvtx_pop();
        if (!on || used >= 4096) return;
        cudaEventRecord(recs[used].b, st);
        ++used;
    }
    void collect()
    {
        for (int i = 0; i < used; ++i) {
            float t = 0.f;
            if (cudaEventElapsedTime(&t, recs[i].a, recs[i].b) == cudaSuccess) {
                ms[recs[i].kid] += t;
                launches[recs[i].kid] += 1;
            }
        }
        used = 0;
    }
    void reset()
    {
        used = 0;
        for (int i = 0; i < KID_COUNT; ++i) { ms[i] = 0; launches[i] = 0; }
    }
    void destroy()
    {
        for (int i = 0; i < created; ++i) { cudaEventDestroy(recs[i].a); cudaEventDestroy(recs[i].b); }
        created = used = 0;
    }
};

// One-time-per-device guard (kernel attributes such as the dynamic shared-memory limit are per device).
struct DevOnce {
    unsigned long long mask = 0;
    bool first()
    {
        int d = 0;
        cudaGetDevice(&d);
        const unsigned long long b = 1ull << (d & 63);
        if (mask & b) return false;
        mask |= b;
        return true;
    }
};

// Development switches (environment variables HYENAND_FORCE_GENERIC, HYENAND_GENERIC_ROWS, HYENAND_GENERIC_CORE,
// HYENAND_NO_TMA select the older kernel variants for A/B runs and tests).  They are read once, when a plan is
// created, and travel with the plan: a forward call never looks at the environment.
struct Switches {
    bool force_generic, generic_rows, generic_core, no_tma;
    bool nvtx;                        // HYENAND_NVTX: name every kernel launch with an NVTX range
};
Switches read_switches();

// Device allocations of a plan, each between two guard bands of kGuardBytes filled with a fixed byte.  A kernel
// that writes outside its workspace damages a band; guard_damage() counts the damaged bytes (blocking copies
// of the bands to the host).  This stands in for a memory checker on machines where none can run.
constexpr size_t kGuardBytes = 4096;
constexpr int kMaxGuarded = 24;
struct GuardedAllocs {
    struct Rec { unsigned char *base; size_t bytes; };
    Rec recs[kMaxGuarded];
    int n = 0;
};
// cudaMalloc of bytes + two bands; *ptr is the first usable byte (256-byte aligned).  cudaSuccess or the error.
cudaError_t guarded_alloc(GuardedAllocs *g, void **ptr, size_t bytes);
void guarded_free_all(GuardedAllocs *g);
long long guard_damage(const GuardedAllocs *g);       // damaged guard bytes, -1 if a copy failed

constexpr int kMaxLineLog2 = 13;          // longest line transformed in shared memory: 8192 points
constexpr int kThreads = 256;             // threads per CTA of the generic kernels

// ---- generic N-D path (nd_kernels.cu) ---------------------------------------------
//
// Workspace arrays hold half spectra along the contiguous axis: XH = P3/2 + 1
// complex bins per row.  "Rows" are lines along the contiguous axis; all other
// axes are transformed by the axis kernels on tiles of adjacent bins.

struct RowsArgs {
    const void *a;        // k (or h)
    const void *b;        // v (or nullptr: plain copy of a)
    float2 *out;          // [rows][pitch], P/2+1 bins written per row
    int pitch;            // elements between rows of out (even, so rows are 16-byte aligned)
    long long rows;       // number of rows
    int len;              // valid elements per row (L3, or K3 for the filter)
    int shift;            // element m of a row goes to padded position (m - shift) mod P
    int log2p;            // log2 of the padded row length P
    int prune_in;         // 1: all valid positions are < P/2 (u, causal h)
    const float2 *gtw;    // global twiddle table, gtw_n points
    int gtw_n;
    int full_in;          // 1: circular mode, k*v rows fill the whole line (len == P): nothing to prune
};

struct RowsInvArgs {
    const float2 *in;     // [rows][pitch]
    int pitch;
    const void *q;        // [rows][len]; nullptr: no gate
    void *y;              // [rows][len]
    const void *q2;       // optional second gate and result of the same rows: y2 = q2 * rows (both or none; the backward
    void *y2;             // pass: dk = v du and dv = k du leave one kernel, du is never stored)
    long long rows;
    int len;              // L3
    int log2p;
    const float2 *gtw;
    int gtw_n;
    int full_out;         // 1: no output half is cropped away, the first len <= P outputs of a row are kept (circular mode: len == P)
};

// A family of strided lines: line (o, c), element a at base[o*outer + a*nc + c].
struct AxisArgs {
    // u lines (in) -> out lines; for the core, in place (out == in, n_out == n_in)
    const float2 *in;
    float2 *out;
    long long n_outer;        // number of outer indices
    long long in_outer;       // element stride between outer indices (input)
    long long out_outer;      // element stride between outer indices (output)
    int nc;                   // contiguous lines per outer index (= element stride along the axis)
    int n_in;                 // valid input entries along the axis
    int n_out;                // entries written along the axis
    int shift;                // input entry m goes to position (m - shift) mod P
    int log2p;
    int prune_in;
    // core only: filter lines, outer index oh = h_shared ? o % h_mod : o
    const float2 *h;
    long long h_outer;
    int h_n_in;
    int h_shift;
    int h_prune_in;
    long long h_mod;          // 0: oh = o, else oh = (o + h_off) % h_mod
    long long h_off;
    float scale;              // applied to the product (1/P_total)
    const float2 *gtw;
    int gtw_n;
    int full;                 // 1: circular mode (n_in == n_out == P): no pruned input half, all outputs kept
    int h_conj;               // core only, 1: the product takes the conjugate of the filter spectrum (the kernel read at the
                              // opposite displacement, h'[d] = h[-d]: the filter of the backward pass's input gradient)
};

enum AxisMode { AXIS_FWD = 0, AXIS_INV = 1, AXIS_CORE = 2 };

int launch_rows_fwd(const RowsArgs &a, int dtype, cudaStream_t st);
int launch_rows_inv(const RowsInvArgs &a, int dtype, cudaStream_t st);

// warp-engine versions (rows_w.cu) for padded row lengths 64..1024
bool rows_w_supported(int log2p);
int launch_rows_fwd_w(const RowsArgs &a, int dtype, cudaStream_t st);
int launch_rows_inv_w(const RowsInvArgs &a, int dtype, cudaStream_t st);
int launch_axis(const AxisArgs &a, int mode, cudaStream_t st);

// warp-engine version of AXIS_CORE (core_w.cu); needs n_in <= P/2, h_n_in <= P, n_out <= P/2
bool core_w_supported(int log2p);
int launch_core_w(const AxisArgs &a, cudaStream_t st);
// warp-engine version of AXIS_FWD / AXIS_INV for 64- to 1024-point axes (core_w.cu); -1 where it does not apply
int launch_axis_w(const AxisArgs &a, bool inverse, cudaStream_t st);

}  // namespace hn
