"""CPU oracle for the gated N-D long convolution -- TEST INFRASTRUCTURE ONLY.

Thin ctypes front end over ``hyenand_oracle.c`` (plain C, fp64, OpenMP over
independent outputs).  It exists so the tests, the smoke check and the
benchmark's CPU-baseline leg can compute the operator of Definition A.3 /
Eq. 1-2 of the paper without touching the CUDA library.  Nothing in the
product package may import this module, and this module imports nothing from
the product package.

Arguments are array-likes (numpy arrays or CPU torch tensors of any float
dtype, bfloat16 included); they are widened exactly to float64 before use.

    q, k, v : [B, C, L_1, ..., L_N]
    h       : [B, C, K_1, ..., K_N]  or  [C, K_1, ..., K_N] (shared over the batch)
    mode    : "linear"   K_n = 2 L_n - 1, tap index = displacement + L_n - 1
              "causal"   N = 1, K_1 = L_1, tap index = displacement >= 0
              "circular" K_n = L_n, tap index = displacement mod L_n
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "hyenand_oracle.c")
_LIB = os.path.join(_HERE, "libhyenand_oracle.so")
_MODES = {"linear": 0, "causal": 1, "circular": 2}
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP); returns the library path."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-std=gnu11", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        dp = ctypes.POINTER(ctypes.c_double)
        ip = ctypes.POINTER(ctypes.c_int)
        llp = ctypes.POINTER(ctypes.c_longlong)
        common = [ctypes.c_int, ip, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                  dp, dp, dp, dp, ctypes.c_longlong]
        lib.hn_oracle_direct.argtypes = common + [dp]
        lib.hn_oracle_fft.argtypes = common + [dp]
        lib.hn_oracle_direct_at.argtypes = common + [ctypes.c_longlong, llp, dp]
        lib.hn_oracle_fftn.argtypes = [ctypes.c_int, ip, dp, ctypes.c_int]
        lib.hn_oracle_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def threads() -> int:
    """Number of OpenMP threads the oracle uses."""
    return int(_load().hn_oracle_threads())


def to_f64(x) -> np.ndarray:
    """Exact widening of any float array-like (bf16 torch tensors included)."""
    if hasattr(x, "detach"):                       # torch tensor, without importing torch
        x = x.detach().cpu().double().numpy()
    return np.ascontiguousarray(np.asarray(x, dtype=np.float64))


def _dp(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def _prep(q, k, v, h, mode):
    q, k, v, h = (to_f64(t) for t in (q, k, v, h))
    if q.shape != k.shape or q.shape != v.shape or q.ndim < 3:
        raise ValueError("q, k, v must share a [B, C, L_1..L_N] shape")
    B, C = q.shape[:2]
    dims = q.shape[2:]
    ndim = len(dims)
    m = _MODES[mode]
    taps = tuple((2 * L - 1) if m == 0 else L for L in dims)
    if h.shape == (C,) + taps:
        hstride = 0
    elif h.shape == (B, C) + taps:
        hstride = C * int(np.prod(taps))
    else:
        raise ValueError(f"h has shape {h.shape}, expected {(B, C) + taps} or {(C,) + taps}")
    cdims = (ctypes.c_int * ndim)(*dims)
    return q, k, v, h, ndim, cdims, B, C, m, hstride


def _check(code):
    if code != 0:
        raise ValueError({1: "invalid argument", 2: "unsupported mode for these dims",
                          3: "out of memory"}.get(code, f"oracle error {code}"))


def conv_direct(q, k, v, h, mode: str = "linear") -> np.ndarray:
    """O1: the defining sums, whole tensor (cost B*C*L^2)."""
    q, k, v, h, ndim, cdims, B, C, m, hs = _prep(q, k, v, h, mode)
    y = np.empty_like(q)
    _check(_load().hn_oracle_direct(ndim, cdims, B, C, m, _dp(q), _dp(k), _dp(v), _dp(h), hs, _dp(y)))
    return y


def conv_direct_at(q, k, v, h, flat_index, mode: str = "linear") -> np.ndarray:
    """O1 at the given flat positions of the [B, C, L_1..L_N] output (cost L each)."""
    q, k, v, h, ndim, cdims, B, C, m, hs = _prep(q, k, v, h, mode)
    idx = np.ascontiguousarray(np.asarray(flat_index, dtype=np.int64))
    if idx.size and (idx.min() < 0 or idx.max() >= q.size):
        raise ValueError("flat index out of range")
    out = np.empty(idx.shape, dtype=np.float64)
    _check(_load().hn_oracle_direct_at(
        ndim, cdims, B, C, m, _dp(q), _dp(k), _dp(v), _dp(h), hs,
        idx.size, idx.ctypes.data_as(ctypes.POINTER(ctypes.c_longlong)), _dp(out)))
    return out


def conv_fft(q, k, v, h, mode: str = "linear") -> np.ndarray:
    """O2: zero-pad, radix-2 N-D FFT, spectral product, inverse, crop, gate."""
    q, k, v, h, ndim, cdims, B, C, m, hs = _prep(q, k, v, h, mode)
    y = np.empty_like(q)
    _check(_load().hn_oracle_fft(ndim, cdims, B, C, m, _dp(q), _dp(k), _dp(v), _dp(h), hs, _dp(y)))
    return y


def fftn(x, inverse: bool = False) -> np.ndarray:
    """The oracle's own unnormalised N-D radix-2 transform (power-of-two axes)."""
    x = np.ascontiguousarray(np.asarray(x, dtype=np.complex128))
    P = (ctypes.c_int * x.ndim)(*x.shape)
    out = x.copy()
    _check(_load().hn_oracle_fftn(x.ndim, P, out.ctypes.data_as(ctypes.POINTER(ctypes.c_double)),
                                  1 if inverse else 0))
    return out


def rel_l2(y, y_ref) -> float:
    """Relative L2 error over the whole tensor against the unrounded fp64 reference."""
    y = to_f64(y)
    y_ref = to_f64(y_ref)
    return float(np.linalg.norm((y - y_ref).ravel()) / max(np.linalg.norm(y_ref.ravel()), 1e-300))
