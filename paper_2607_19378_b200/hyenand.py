"""ctypes binding of libhyenand.so: argument marshalling only.

Every function has the name and meaning of the C entry point declared in
include/hyenand.h; tensors are passed as raw device (or host) pointers and all
arithmetic happens in the library's CUDA kernels.  There is no fallback: if the
library has not been built, loading raises.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# HYENAND_LIB=debug selects the checked build (libhyenand_debug.so, see hyenand_debug_build in the header)
LIB_PATH = os.path.join(_HERE, "libhyenand_debug.so" if os.environ.get("HYENAND_LIB") == "debug" else "libhyenand.so")

HYENAND_F32 = 0
HYENAND_BF16 = 1
HYENAND_MODE_LINEAR = 0
HYENAND_MODE_CAUSAL = 1
HYENAND_MODE_CIRCULAR = 2
HYENAND_OK = 0
HYENAND_ERR_INVALID_ARG = 1
HYENAND_ERR_UNSUPPORTED = 2
HYENAND_ERR_ALLOC = 3
HYENAND_ERR_CUDA = 4

_DTYPES = {torch.float32: HYENAND_F32, torch.bfloat16: HYENAND_BF16}
_lib = None


class HyenaNDError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"hyenand error {code}: {msg}")
        self.code = code


def lib() -> ctypes.CDLL:
    """The loaded C library (raises if it was never built)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise OSError(f"{LIB_PATH} is missing: build it with `python -m paper_2607_19378_b200.build`")
        L = ctypes.CDLL(LIB_PATH)
        vp, ip, ll = ctypes.c_void_p, ctypes.POINTER(ctypes.c_int), ctypes.c_longlong
        L.hyenand_create_plan.restype = vp
        L.hyenand_create_plan.argtypes = [ctypes.c_int, ip, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int]
        L.hyenand_create_plan_mode.restype = vp
        L.hyenand_create_plan_mode.argtypes = [ctypes.c_int, ip, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int]
        L.hyenand_forward.argtypes = [vp, vp, vp, vp, vp, vp, vp]
        L.hyenand_forward_ex.argtypes = [vp, vp, vp, vp, vp, ll, vp, vp]
        L.hyenand_forward_host.argtypes = [vp, vp, vp, vp, vp, ll, vp, vp]
        L.hyenand_destroy_plan.argtypes = [vp]
        L.hyenand_destroy_plan.restype = None
        L.hyenand_last_error.restype = ctypes.c_char_p
        L.hyenand_debug_build.restype = ctypes.c_int
        L.hyenand_debug_violations.restype = ll
        L.hyenand_debug_violations.argtypes = [ctypes.POINTER(ctypes.c_ulonglong), ip, ctypes.POINTER(ctypes.c_char_p)]
        L.hyenand_debug_selftest.restype = ll
        L.hyenand_synth_device_status.restype = ctypes.c_int
        L.hyenand_selftest_bounded_wait.argtypes = [ctypes.c_int]
        L.hyenand_selftest_bounded_wait.restype = ctypes.c_int
        L.hyenand_plan_device_status.argtypes = [vp]
        L.hyenand_plan_device_status.restype = ctypes.c_int
        L.hyenand_plan_workspace_bytes.argtypes = [vp]
        L.hyenand_plan_workspace_bytes.restype = ctypes.c_size_t
        L.hyenand_plan_fft_dims.argtypes = [vp, ip]
        L.hyenand_plan_launches.argtypes = [vp, ctypes.c_int]
        L.hyenand_plan_path.argtypes = [vp]
        L.hyenand_plan_path.restype = ctypes.c_char_p
        L.hyenand_plan_groups.argtypes = [vp, ctypes.POINTER(ll), ip]
        L.hyenand_plan_guard_damage.argtypes = [vp]
        L.hyenand_plan_guard_damage.restype = ll
        dpp = ctypes.POINTER(ctypes.c_double)
        L.hyenand_plan_kernel_count.argtypes = [vp]
        L.hyenand_plan_kernel_info.argtypes = [vp, ctypes.c_int, ctypes.c_int, ctypes.POINTER(ctypes.c_char_p),
                                               dpp, dpp, dpp]
        L.hyenand_noalloc_max_bytes.restype = ctypes.c_size_t
        L.hyenand_forward_noalloc.argtypes = [ctypes.c_int, ip, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                              vp, vp, vp, vp, ll, vp, vp]
        fp = ctypes.POINTER(ctypes.c_float)
        L.hyenand_mixer_create.restype = vp
        L.hyenand_mixer_create.argtypes = [ctypes.c_int, ip, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_float]
        L.hyenand_mixer_forward.argtypes = [vp, vp, vp, vp, vp, ll, vp, vp, vp, vp]
        L.hyenand_mixer_plan.restype = vp
        L.hyenand_mixer_plan.argtypes = [vp]
        L.hyenand_mixer_guard_damage.restype = ll
        L.hyenand_mixer_guard_damage.argtypes = [vp]
        L.hyenand_mixer_destroy.restype = None
        L.hyenand_mixer_destroy.argtypes = [vp]
        L.hyenand_backward_create.restype = vp
        L.hyenand_backward_create.argtypes = [ctypes.c_int, ip, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int]
        L.hyenand_backward.argtypes = [vp, vp, vp, vp, vp, ll, vp, vp, vp, vp, vp, vp]
        L.hyenand_backward_guard_damage.restype = ll
        L.hyenand_backward_guard_damage.argtypes = [vp]
        L.hyenand_backward_destroy.restype = None
        L.hyenand_backward_destroy.argtypes = [vp]
        L.hyenand_synthesize_kernel.argtypes = [ctypes.c_int, ip] + [ctypes.c_int] * 5 + [vp] * 10 + [ctypes.c_int, vp, vp]
        L.hyenand_plan_set_timing.argtypes = [vp, ctypes.c_int]
        L.hyenand_plan_kernel_time.argtypes = [vp, ctypes.c_int, dpp, dpp]
        _lib = L
    return _lib


def hyenand_last_error() -> str:
    return lib().hyenand_last_error().decode()


def hyenand_last_error_code() -> int:
    return int(lib().hyenand_last_error_code())


def _check(code: int):
    if code != HYENAND_OK:
        raise HyenaNDError(code, hyenand_last_error())


def hyenand_create_plan(ndim: int, dims, B: int, C: int, causal: int, dtype: int) -> int:
    arr = (ctypes.c_int * max(1, len(dims)))(*[int(d) for d in dims])
    h = lib().hyenand_create_plan(int(ndim), arr, int(B), int(C), int(causal), int(dtype))
    if not h:
        msg = hyenand_last_error()
        code = hyenand_last_error_code() or HYENAND_ERR_INVALID_ARG
        raise HyenaNDError(code, msg)
    return h


def hyenand_create_plan_mode(ndim: int, dims, B: int, C: int, mode: int, dtype: int) -> int:
    arr = (ctypes.c_int * max(1, len(dims)))(*[int(d) for d in dims])
    h = lib().hyenand_create_plan_mode(int(ndim), arr, int(B), int(C), int(mode), int(dtype))
    if not h:
        msg = hyenand_last_error()
        code = hyenand_last_error_code() or HYENAND_ERR_INVALID_ARG
        raise HyenaNDError(code, msg)
    return h


def hyenand_destroy_plan(plan: int) -> None:
    lib().hyenand_destroy_plan(plan)


def _stream_ptr(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream) if hasattr(stream, "cuda_stream") else int(stream)


def hyenand_forward(plan: int, q, k, v, h, y, stream=None) -> None:
    _check(lib().hyenand_forward(plan, q.data_ptr(), k.data_ptr(), v.data_ptr(), h.data_ptr(),
                                 y.data_ptr(), _stream_ptr(stream)))


def hyenand_forward_ex(plan: int, q, k, v, h, h_batch_stride_elems: int, y, stream=None) -> None:
    _check(lib().hyenand_forward_ex(plan, q.data_ptr(), k.data_ptr(), v.data_ptr(), h.data_ptr(),
                                    int(h_batch_stride_elems), y.data_ptr(), _stream_ptr(stream)))


def hyenand_forward_host(plan: int, q, k, v, h, h_batch_stride_elems: int, y, stream=None) -> None:
    _check(lib().hyenand_forward_host(plan, q.data_ptr(), k.data_ptr(), v.data_ptr(), h.data_ptr(),
                                      int(h_batch_stride_elems), y.data_ptr(), _stream_ptr(stream)))


def hyenand_debug_build() -> bool:
    return bool(lib().hyenand_debug_build())


def hyenand_debug_violations():
    """(count, first address, first line, first file) of the checked build's out-of-range accesses since the last call;
    count is -1 in the product library."""
    addr, line, name = ctypes.c_ulonglong(), ctypes.c_int(), ctypes.c_char_p()
    n = lib().hyenand_debug_violations(ctypes.byref(addr), ctypes.byref(line), ctypes.byref(name))
    return int(n), int(addr.value), int(line.value), (name.value or b"").decode()


def hyenand_synth_device_status() -> int:
    return int(lib().hyenand_synth_device_status())


def hyenand_debug_selftest() -> int:
    return int(lib().hyenand_debug_selftest())


def hyenand_selftest_bounded_wait(polls: int = 1000) -> int:
    """9 if a wait on a barrier that nothing completes ran out and was reported, as it must."""
    return int(lib().hyenand_selftest_bounded_wait(int(polls)))


def hyenand_plan_device_status(plan: int) -> int:
    """0 unless a kernel of the plan gave up a bounded wait (synchronise the stream first)."""
    return int(lib().hyenand_plan_device_status(plan))


def hyenand_plan_workspace_bytes(plan: int) -> int:
    return int(lib().hyenand_plan_workspace_bytes(plan))


def hyenand_plan_fft_dims(plan: int, ndim: int):
    out = (ctypes.c_int * ndim)()
    _check(lib().hyenand_plan_fft_dims(plan, out))
    return tuple(out)


def hyenand_plan_launches(plan: int, h_shared: bool) -> int:
    return int(lib().hyenand_plan_launches(plan, 1 if h_shared else 0))


def hyenand_plan_path(plan: int) -> str:
    return lib().hyenand_plan_path(plan).decode()


def hyenand_plan_groups(plan: int):
    """(slices per group, lanes): how one forward schedules the batch."""
    n, lanes = ctypes.c_longlong(), ctypes.c_int()
    _check(lib().hyenand_plan_groups(plan, ctypes.byref(n), ctypes.byref(lanes)))
    return int(n.value), int(lanes.value)


def hyenand_plan_guard_damage(plan: int) -> int:
    """Bytes of the guard bands around the plan's device allocations that a kernel overwrote (0 = none)."""
    return int(lib().hyenand_plan_guard_damage(plan))


def hyenand_plan_kernel_count(plan: int) -> int:
    return int(lib().hyenand_plan_kernel_count(plan))


def hyenand_plan_kernel_info(plan: int, kernel_id: int, h_shared: bool):
    """(name, launches, algorithmic bytes, algorithmic flops) of one kernel, per forward."""
    name = ctypes.c_char_p()
    n, b, f = ctypes.c_double(), ctypes.c_double(), ctypes.c_double()
    _check(lib().hyenand_plan_kernel_info(plan, kernel_id, 1 if h_shared else 0, ctypes.byref(name),
                                          ctypes.byref(n), ctypes.byref(b), ctypes.byref(f)))
    return name.value.decode(), n.value, b.value, f.value


def hyenand_plan_set_timing(plan: int, enable) -> None:
    """0/False: off; 1/True: time every launch; 2: the same with the plan's lanes run one after the other."""
    _check(lib().hyenand_plan_set_timing(plan, int(enable)))


def hyenand_plan_kernel_time(plan: int, kernel_id: int):
    """(accumulated device ms, recorded launches) since timing was switched on."""
    ms, n = ctypes.c_double(), ctypes.c_double()
    _check(lib().hyenand_plan_kernel_time(plan, kernel_id, ctypes.byref(ms), ctypes.byref(n)))
    return ms.value, n.value


def hyenand_noalloc_max_bytes() -> int:
    return int(lib().hyenand_noalloc_max_bytes())


def hyenand_forward_noalloc(dims, B: int, C: int, causal: int, dtype: int, q, k, v, h,
                            h_batch_stride_elems: int, y, stream=None) -> None:
    """Forward through the entry point that allocates no device memory (fixed workspace inside
    the library; see include/hyenand.h for its limits and the rule about overlapping calls)."""
    arr = (ctypes.c_int * max(1, len(dims)))(*[int(d) for d in dims])
    _check(lib().hyenand_forward_noalloc(len(dims), arr, int(B), int(C), int(causal), int(dtype),
                                         q.data_ptr(), k.data_ptr(), v.data_ptr(), h.data_ptr(),
                                         int(h_batch_stride_elems), y.data_ptr(), _stream_ptr(stream)))


def hyenand_mixer_create(ndim: int, dims, B: int, C: int, mode: int, dtype: int, eps: float) -> int:
    arr = (ctypes.c_int * max(1, len(dims)))(*[int(d) for d in dims])
    h = lib().hyenand_mixer_create(int(ndim), arr, int(B), int(C), int(mode), int(dtype), float(eps))
    if not h:
        raise HyenaNDError(hyenand_last_error_code() or HYENAND_ERR_INVALID_ARG, hyenand_last_error())
    return h


def hyenand_mixer_forward(mixer: int, q, k, v, h, h_batch_stride_elems: int, g_in, g_out, y, stream=None) -> None:
    _check(lib().hyenand_mixer_forward(mixer, q.data_ptr(), k.data_ptr(), v.data_ptr(), h.data_ptr(),
                                       int(h_batch_stride_elems), g_in.data_ptr(), g_out.data_ptr(), y.data_ptr(),
                                       _stream_ptr(stream)))


def hyenand_mixer_plan(mixer: int) -> int:
    return lib().hyenand_mixer_plan(mixer)


def hyenand_mixer_guard_damage(mixer: int) -> int:
    return int(lib().hyenand_mixer_guard_damage(mixer))


def hyenand_mixer_destroy(mixer: int) -> None:
    lib().hyenand_mixer_destroy(mixer)


def hyenand_synthesize_kernel(dims, mode: int, B: int, C: int, hidden: int, layers: int, W1, b1, omega0, Wh, bh, Wout,
                              bout, gamma, beta, window, dtype: int, h, stream=None) -> None:
    """K(x) on the tap grid of `dims` into h (device tensor [B, C, K..]); parameters: fp32 device tensors, gamma and
    beta may both be None (static kernel), Wh and bh may be None when layers == 1."""
    arr = (ctypes.c_int * max(1, len(dims)))(*[int(d) for d in dims])
    ptr = lambda t: None if t is None else t.data_ptr()
    _check(lib().hyenand_synthesize_kernel(len(dims), arr, int(mode), int(B), int(C), int(hidden), int(layers),
                                           ptr(W1), ptr(b1), ptr(omega0), ptr(Wh), ptr(bh), ptr(Wout), ptr(bout),
                                           ptr(gamma), ptr(beta), ptr(window), int(dtype), h.data_ptr(), _stream_ptr(stream)))


def hyenand_backward_create(ndim: int, dims, B: int, C: int, mode: int, dtype: int) -> int:
    arr = (ctypes.c_int * max(1, len(dims)))(*[int(d) for d in dims])
    h = lib().hyenand_backward_create(int(ndim), arr, int(B), int(C), int(mode), int(dtype))
    if not h:
        raise HyenaNDError(hyenand_last_error_code() or HYENAND_ERR_INVALID_ARG, hyenand_last_error())
    return h


def hyenand_backward(grad: int, q, k, v, h, h_batch_stride_elems: int, dy, dq, dk, dv, dh, stream=None) -> None:
    _check(lib().hyenand_backward(grad, q.data_ptr(), k.data_ptr(), v.data_ptr(), h.data_ptr(), int(h_batch_stride_elems),
                                  dy.data_ptr(), dq.data_ptr(), dk.data_ptr(), dv.data_ptr(), dh.data_ptr(), _stream_ptr(stream)))


def hyenand_backward_guard_damage(grad: int) -> int:
    return int(lib().hyenand_backward_guard_damage(grad))


def hyenand_backward_destroy(grad: int) -> None:
    lib().hyenand_backward_destroy(grad)


class Backward:
    """Owner of a hyenand_grad handle: dq, dk, dv, dh of the gated long convolution."""

    def __init__(self, dims, B: int, C: int, mode: str = "linear", dtype=torch.float32):
        self.dims = tuple(int(d) for d in dims)
        self.B, self.C, self.mode, self.dtype = B, C, mode, dtype
        code = {"linear": HYENAND_MODE_LINEAR, "causal": HYENAND_MODE_CAUSAL, "circular": HYENAND_MODE_CIRCULAR}[mode]
        self.handle = hyenand_backward_create(len(self.dims), self.dims, B, C, code, _DTYPES[dtype])

    def __call__(self, q, k, v, h, dy, stream=None):
        taps = tuple(2 * L - 1 if self.mode == "linear" else L for L in self.dims)
        if tuple(h.shape) == (self.C,) + taps:
            stride = 0
        elif tuple(h.shape) == (self.B, self.C) + taps:
            stride = self.C * h[0, 0].numel()
        else:
            raise ValueError(f"h has shape {tuple(h.shape)}")
        for t in (q, k, v, h, dy):
            if not (t.is_cuda and t.is_contiguous() and t.dtype == self.dtype):
                raise ValueError("inputs must be contiguous CUDA tensors of the handle's dtype")
        dq, dk, dv, dh = torch.empty_like(q), torch.empty_like(q), torch.empty_like(q), torch.empty_like(h)
        hyenand_backward(self.handle, q, k, v, h, stride, dy, dq, dk, dv, dh, stream)
        return dq, dk, dv, dh

    def close(self):
        if self.handle:
            hyenand_backward_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class Mixer:
    """Owner of a hyenand_mixer handle: the full operator of Eq. 2 (pointwise stages + long convolution)."""

    def __init__(self, dims, B: int, C: int, mode: str = "linear", dtype=torch.float32, eps: float = 1e-6):
        self.dims = tuple(int(d) for d in dims)
        self.B, self.C, self.mode, self.dtype = B, C, mode, dtype
        code = {"linear": HYENAND_MODE_LINEAR, "causal": HYENAND_MODE_CAUSAL, "circular": HYENAND_MODE_CIRCULAR}[mode]
        self.handle = hyenand_mixer_create(len(self.dims), self.dims, B, C, code, _DTYPES[dtype], eps)

    def forward(self, q, k, v, h, g_in, g_out, y=None, stream=None):
        taps = tuple(2 * L - 1 if self.mode == "linear" else L for L in self.dims)
        if tuple(h.shape) == (self.C,) + taps:
            stride = 0
        elif tuple(h.shape) == (self.B, self.C) + taps:
            stride = self.C * h[0, 0].numel()
        else:
            raise ValueError(f"h has shape {tuple(h.shape)}")
        for t in (q, k, v, h):
            if not (t.is_cuda and t.is_contiguous() and t.dtype == self.dtype):
                raise ValueError("inputs must be contiguous CUDA tensors of the mixer's dtype")
        for g in (g_in, g_out):
            if not (g.is_cuda and g.is_contiguous() and g.dtype == torch.float32 and g.numel() == self.C):
                raise ValueError("g_in, g_out must be contiguous fp32 CUDA tensors of C elements")
        if y is None:
            y = torch.empty_like(q)
        hyenand_mixer_forward(self.handle, q, k, v, h, stride, g_in, g_out, y, stream)
        return y

    def close(self):
        if self.handle:
            hyenand_mixer_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class Plan:
    """Convenience owner of a plan handle (create on construction, destroy on close)."""

    def __init__(self, dims, B: int, C: int, causal: bool = False, dtype=torch.float32, circular: bool = False):
        self.dims = tuple(int(d) for d in dims)
        self.B, self.C, self.causal, self.dtype, self.circular = B, C, bool(causal), dtype, bool(circular)
        if self.circular:
            if self.causal:
                raise ValueError("a plan is causal or circular, not both")
            self.handle = hyenand_create_plan_mode(len(self.dims), self.dims, B, C, HYENAND_MODE_CIRCULAR, _DTYPES[dtype])
        else:
            self.handle = hyenand_create_plan(len(self.dims), self.dims, B, C, int(self.causal), _DTYPES[dtype])

    def _stride(self, h) -> int:
        taps = tuple(L if (self.causal or self.circular) else 2 * L - 1 for L in self.dims)
        if tuple(h.shape) == (self.C,) + taps:
            return 0
        if tuple(h.shape) == (self.B, self.C) + taps:
            return self.C * h[0, 0].numel()
        raise ValueError(f"h has shape {tuple(h.shape)}")

    def forward(self, q, k, v, h, y=None, stream=None):
        """Device tensors in, device tensor out (enqueued on the current stream)."""
        for t in (q, k, v, h):
            if not (t.is_cuda and t.is_contiguous() and t.dtype == self.dtype):
                raise ValueError("inputs must be contiguous CUDA tensors of the plan's dtype")
        if y is None:
            y = torch.empty_like(q)
        hyenand_forward_ex(self.handle, q, k, v, h, self._stride(h), y, stream)
        return y

    def forward_host(self, q, k, v, h, y, stream=None):
        """Host tensors in, host tensor out; copies run inside the call."""
        hyenand_forward_host(self.handle, q, k, v, h, self._stride(h), y, stream)
        return y

    @property
    def launches_per_forward(self):
        return lambda shared: hyenand_plan_launches(self.handle, shared)

    def close(self):
        if self.handle:
            hyenand_destroy_plan(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
