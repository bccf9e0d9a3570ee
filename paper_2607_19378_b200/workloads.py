"""Seeded synthetic inputs for the gated N-D long convolution.

This module only draws numbers: it holds none of the operator's arithmetic and
is the one piece of code that both the CUDA path's callers and the CPU oracle's
callers use, so that both sides consume identical arrays.  Tensors are built
with torch on whatever device is asked for (the CPU for small cases; the GPU
for the full-size workloads, copied back to the host for the oracle).

The five named workloads stand in for the workloads the paper evaluates on
(its datasets are not needed: the operator's cost does not depend on values):

    tiny2d      2-D 32x32, fp32, one filter per (b, c), L1-decaying filter
    genomics1d  causal 1-D, L = 262144, bf16, one filter per channel
                (long-context genomics layer, Section 5.2 / Appendix B.3)
    vision2d    2-D 64x64 token grid, bf16, one filter per (b, c)
                (ImageNet / spatial-recall token grids, Section 5.1, 5.3)
    pde2d       2-D 512x512 smooth fields, fp32 (The Well, Section 5.4)
    volume3d    3-D 128^3, bf16 (medical volumes, Section 5.5)

Filters decay away from displacement zero the way the windowed kernels of
Section 3.2.1 / Appendix A.3 do (exponential window for the causal 1-D case,
radially decaying windows otherwise).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, replace
from typing import Tuple

import torch


@dataclass(frozen=True)
class Workload:
    name: str
    dims: Tuple[int, ...]
    B: int
    C: int
    dtype: str            # "f32" | "bf16"  (I/O type of q, k, v, h, y)
    causal: bool = False
    h_shared: bool = False  # one filter per channel, shared by the batch
    seed: int = 0
    filt: str = "radial"  # "l1" | "causal_exp" | "radial" | "spectral"
    alpha: Tuple[float, float] = (0.05, 1.0)
    field: str = "normal"  # "normal" | "spectral"
    circular: bool = False  # periodic boundaries: the filter lives on the grid itself (K_n = L_n)

    @property
    def ndim(self) -> int:
        return len(self.dims)

    @property
    def taps(self) -> Tuple[int, ...]:
        return tuple(L if (self.causal or self.circular) else 2 * L - 1 for L in self.dims)

    @property
    def mode(self) -> str:
        """Boundary handling in the oracle's vocabulary."""
        return "causal" if self.causal else "circular" if self.circular else "linear"

    @property
    def elements(self) -> int:
        return self.B * self.C * math.prod(self.dims)

    @property
    def torch_dtype(self) -> torch.dtype:
        return torch.float32 if self.dtype == "f32" else torch.bfloat16

    def scaled(self, B: int | None = None, C: int | None = None) -> "Workload":
        """Same shapes per slice with fewer (or more) batch entries / channels."""
        return replace(self, B=self.B if B is None else B, C=self.C if C is None else C)


WORKLOADS = {
    "tiny2d": Workload("tiny2d", (32, 32), 1, 8, "f32", seed=0, filt="l1"),
    "genomics1d": Workload("genomics1d", (262144,), 2, 256, "bf16", causal=True, h_shared=True,
                           seed=2, filt="causal_exp", alpha=(0.5, 8.0)),
    "vision2d": Workload("vision2d", (64, 64), 16, 768, "bf16", seed=3, filt="radial",
                         alpha=(0.05, 1.0)),
    "pde2d": Workload("pde2d", (512, 512), 4, 128, "f32", seed=4, filt="spectral", field="spectral"),
    "volume3d": Workload("volume3d", (128, 128, 128), 1, 64, "bf16", seed=5, filt="radial",
                         alpha=(0.05, 0.5)),
}

# Workloads of the rows built after the five above (not part of the default benchmark table):
#   periodic2d  2-D 512x512 smooth fields with periodic boundaries, fp32: the circular mode of Section 3.2.1,
#               shaped like the periodic PDE fields of Section 5.4
EXTRA_WORKLOADS = {
    "periodic2d": Workload("periodic2d", (512, 512), 4, 128, "f32", seed=6, filt="radial", alpha=(0.02, 0.3),
                           field="spectral", circular=True),
}


def _gen(seed: int, stream: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed * 1000003 + stream)
    return g


def _normal(shape, g, device):
    return torch.randn(shape, generator=g, device=device, dtype=torch.float32)


def _smooth_field(shape, g, device):
    """Gaussian noise low-passed with spectral decay |kappa|^-2 (zero mean, unit variance)."""
    *lead, n1, n2 = shape
    noise = _normal(shape, g, device)
    spec = torch.fft.rfft2(noise)
    k1 = torch.fft.fftfreq(n1, device=device) * n1
    k2 = torch.fft.rfftfreq(n2, device=device) * n2
    kap2 = k1[:, None] ** 2 + k2[None, :] ** 2
    w = torch.where(kap2 > 0, 1.0 / kap2.clamp_min(1.0), torch.zeros_like(kap2))
    out = torch.fft.irfft2(spec * w, s=(n1, n2))
    out = out - out.mean(dim=(-2, -1), keepdim=True)
    out = out / out.std(dim=(-2, -1), keepdim=True).clamp_min(1e-20)
    return out


def _offsets(L, causal, device, circular=False):
    if causal:
        return torch.arange(L, device=device, dtype=torch.float32)
    if circular:
        # tap m is the displacement m mod L: its length on the periodic grid is min(m, L - m)
        m = torch.arange(L, device=device, dtype=torch.float32)
        return torch.minimum(m, L - m)
    return torch.arange(-(L - 1), L, device=device, dtype=torch.float32)


def make_filter(w: Workload, device="cpu") -> torch.Tensor:
    """h in the I/O dtype: [C, K..] when shared over the batch, else [B, C, K..]."""
    lead = (w.C,) if w.h_shared else (w.B, w.C)
    g = _gen(w.seed, 4, device)
    ga = _gen(w.seed, 5, device)
    alpha = torch.rand((w.C,), generator=ga, device=device) * (w.alpha[1] - w.alpha[0]) + w.alpha[0]
    alpha = alpha.reshape((w.C,) + (1,) * w.ndim)
    offs = [_offsets(L, w.causal, device, w.circular) for L in w.dims]
    if w.filt == "spectral":
        # same low-passed construction as the fields, built on the padded torus and cropped
        P = tuple(2 * L for L in w.dims)
        out = torch.empty(lead + w.taps, device=device, dtype=torch.float32)
        flat = out.view((-1,) + w.taps)
        for s in range(flat.shape[0]):
            f = _smooth_field(P, g, device)
            flat[s] = f[tuple(slice(0, K) for K in w.taps)]
        h = out
    else:
        if w.filt == "l1":
            dist = sum(o.abs().reshape([-1 if a == i else 1 for a in range(w.ndim)])
                       for i, o in enumerate(offs))
            decay = torch.exp(-0.1 * dist).expand((w.C,) + w.taps)
        elif w.filt == "causal_exp":
            decay = torch.exp(-alpha * offs[0].reshape(1, -1) / float(w.dims[0]))
        else:
            r2 = sum((o ** 2).reshape([-1 if a == i else 1 for a in range(w.ndim)])
                     for i, o in enumerate(offs))
            decay = None  # built per channel below to bound memory
        h = torch.empty(lead + w.taps, device=device, dtype=torch.float32)
        hv = h.view((-1, w.C) + w.taps)
        step = max(1, (1 << 27) // math.prod(w.taps))      # channels per draw, bounds temporaries
        for b in range(hv.shape[0]):
            for c0 in range(0, w.C, step):
                c1 = min(w.C, c0 + step)
                n = _normal((c1 - c0,) + w.taps, g, device)
                d = torch.exp(-alpha[c0:c1] * torch.sqrt(r2)) if decay is None else decay[c0:c1]
                hv[b, c0:c1] = n * d
    h = torch.where(h.abs() < 1e-30, torch.zeros_like(h), h)   # no subnormals on either side
    return h.to(w.torch_dtype).contiguous()


def make_inputs(w: Workload, device="cpu"):
    """(q, k, v, h) in the workload's I/O dtype, dense row-major on `device`."""
    shape = (w.B, w.C) + w.dims
    out = []
    for stream in (1, 2, 3):
        g = _gen(w.seed, stream, device)
        if w.field == "spectral":
            t = _smooth_field(shape, g, device)
        else:
            t = _normal(shape, g, device)
        out.append(t.to(w.torch_dtype).contiguous())
    q, k, v = out
    return q, k, v, make_filter(w, device)


def random_problem(dims, B=2, C=3, dtype="f32", causal=False, h_shared=False, seed=0, device="cpu", circular=False):
    """A small problem of arbitrary shape with N(0,1) inputs and a radially decaying filter."""
    w = Workload("random", tuple(int(d) for d in dims), B, C, dtype, causal=causal,
                 h_shared=h_shared, seed=seed,
                 filt="causal_exp" if causal else "radial", alpha=(0.05, 1.0), circular=circular)
    return w, make_inputs(w, device)
