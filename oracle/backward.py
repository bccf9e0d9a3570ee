"""CPU oracle of the backward pass of the gated long convolution -- TEST INFRASTRUCTURE ONLY.

Forward (Definition A.3 of the paper): y_i = q_i * w_i,  w_i = sum_j h[i - j] u_j,  u = k * v.
Given dy (same shape as y), with g = dy * q the gradient arriving at w:

    dq_i = dy_i * w_i
    du_j = sum_i h[i - j] g_i            (the transpose of the convolution: the kernel read at the opposite displacement)
    dk   = du * v,   dv = du * k
    dh[d] = sum_i g_i u_{i - d}          for every displacement d the kernel has a tap for (summed over the batch as
                                         well when one kernel serves the whole batch)

in float64.  du and w use the convolution oracle (hyenand_oracle.c) with the kernel re-indexed to the opposite
displacement; dh is the sum above, written as loops over the taps (`direct=True`, small cases) or as a correlation
through numpy's FFT on a grid large enough to hold every displacement without wrap-around (`direct=False`).
The paper gives no backward pass (its benchmarks are forward only, Appendix B.4); this is the derivative of its
forward definition, nothing else.
"""
from __future__ import annotations

import numpy as np

from . import conv_direct, conv_fft, to_f64


def opposite_kernel(h: np.ndarray, dims, mode: str):
    """The kernel h'[d] = h[-d] and the mode under which the convolution oracle applies it."""
    nd = len(dims)
    axes = tuple(range(h.ndim - nd, h.ndim))
    if mode == "linear":
        return np.flip(h, axis=axes).copy(), "linear"
    if mode == "circular":
        out = h
        for a in axes:
            out = np.roll(np.flip(out, axis=a), 1, axis=a)      # index m -> (-m) mod L
        return out.copy(), "circular"
    # causal: taps at displacements 0..L-1 move to 0..-(L-1); as a non-causal kernel array over -(L-1)..L-1
    L = dims[0]
    lin = np.zeros(h.shape[:-1] + (2 * L - 1,))
    lin[..., :L] = h[..., ::-1]                                  # array index m = d + L - 1, d = -(L-1)..0
    return lin, "linear"


def tap_displacements(L: int, mode: str) -> np.ndarray:
    if mode == "linear":
        return np.arange(-(L - 1), L)
    return np.arange(L)                                          # causal: d = tap; circular: d = tap (mod L)


def _dh_direct(g, u, dims, mode, taps):
    """dh[d] = sum_i g_i u_{i-d}, one slice ([L..] arrays), by definition."""
    nd = len(dims)
    out = np.zeros(taps)
    disp = [tap_displacements(L, mode) for L in dims]
    for m in np.ndindex(*taps):
        d = [int(disp[a][m[a]]) for a in range(nd)]
        if mode == "circular":
            out[m] = np.sum(g * np.roll(u, shift=d, axis=tuple(range(nd))))      # roll(u, d)[i] = u[(i - d) mod L]
        else:
            gi, ui = [], []
            for a in range(nd):
                lo, hi = max(0, d[a]), min(dims[a], dims[a] + d[a])
                gi.append(slice(lo, hi))
                ui.append(slice(lo - d[a], hi - d[a]))
            out[m] = np.sum(g[tuple(gi)] * u[tuple(ui)])
    return out


def _dh_fft(g, u, dims, mode, taps):
    nd = len(dims)
    P = tuple(L if mode == "circular" else 2 * L for L in dims)
    axes = tuple(range(nd))
    corr = np.fft.irfftn(np.fft.rfftn(g, s=P, axes=axes) * np.conj(np.fft.rfftn(u, s=P, axes=axes)), s=P, axes=axes)
    idx = np.ix_(*[tap_displacements(L, mode) % Pn for L, Pn in zip(dims, P)])
    return corr[idx]


def backward(q, k, v, h, dy, mode: str = "linear", direct: bool = False):
    """(dq, dk, dv, dh) for [B, C, L_1..L_N] tensors; h and dh are [B, C, K..] or [C, K..] (kernel shared over the batch)."""
    q, k, v, h, dy = (to_f64(t) for t in (q, k, v, h, dy))
    B, C = q.shape[:2]
    dims = q.shape[2:]
    nd = len(dims)
    shared = h.ndim == nd + 1
    conv = conv_direct if direct else conv_fft
    one = np.ones_like(q)
    w = conv(one, k, v, h, mode)                                 # the ungated convolution
    dq = dy * w
    g = dy * q
    hopp, opp_mode = opposite_kernel(h, dims, mode)
    du = conv(one, g, one, hopp, opp_mode)
    dk, dv = du * v, du * k
    u = k * v
    taps = h.shape[-nd:]
    dh = np.zeros(h.shape)
    fn = _dh_direct if direct else _dh_fft
    for b in range(B):
        for c in range(C):
            part = fn(g[b, c], u[b, c], dims, mode, taps)
            if shared:
                dh[c] += part
            else:
                dh[b, c] = part
    return dq, dk, dv, dh
