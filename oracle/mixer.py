"""CPU oracle of the full HyenaND operator (Eq. 2 of the paper) -- TEST INFRASTRUCTURE ONLY.

    y = RMSNorm_out( Sigmoid(v) * ( K conv RMSNorm_in( l2(q) * SiLU(k) ) ) )

in plain numpy float64, one statement per step of Eq. 2 in the paper's order (Section 3.2).  The long
convolution is the oracle's own (hyenand_oracle.c: the defining sum, or its radix-2 FFT path); everything
else is written out here.  Channel axis = axis 1 of [B, C, L_1..L_N]; both normalisations act per token
(one grid position of one batch entry) across the C channels.

Readings of the paper where it leaves a constant open (Section 3.2 names the operations, not their epsilons):
  l2(q)      q / max(||q||_2, 1e-12), the norm taken over the channels of a token
  RMSNorm    x / sqrt(mean_c(x^2) + eps) * g, eps inside the root, one learned weight g per channel
  SiLU(k)    k * sigmoid(k);  Sigmoid(v) = 1 / (1 + exp(-v))
"""
from __future__ import annotations

import numpy as np

from . import conv_direct, conv_fft, to_f64

L2_FLOOR = 1e-12


def l2_normalise(q: np.ndarray) -> np.ndarray:
    norm = np.sqrt(np.sum(q * q, axis=1, keepdims=True))
    return q / np.maximum(norm, L2_FLOOR)


def silu(x: np.ndarray) -> np.ndarray:
    return x / (1.0 + np.exp(-x))


def sigmoid(x: np.ndarray) -> np.ndarray:
    return 1.0 / (1.0 + np.exp(-x))


def rms_norm(x: np.ndarray, g: np.ndarray, eps: float) -> np.ndarray:
    ms = np.mean(x * x, axis=1, keepdims=True)
    shape = (1, -1) + (1,) * (x.ndim - 2)
    return x / np.sqrt(ms + eps) * g.reshape(shape)


def hyena_mixer(q, k, v, h, g_in, g_out, eps: float = 1e-6, mode: str = "linear", direct: bool = False,
                parts: bool = False):
    """Eq. 2 on [B, C, L_1..L_N] tensors; h as for the convolution oracle; g_in, g_out: [C].
    parts=True also returns the gated convolution (the argument of the last RMSNorm), for error bounds in tests."""
    q, k, v = (to_f64(t) for t in (q, k, v))
    g_in, g_out = to_f64(g_in), to_f64(g_out)
    inner = l2_normalise(q) * silu(k)                       # l2(q) * SiLU(k)
    z = rms_norm(inner, g_in, eps)                          # RMSNorm before the long convolution
    one = np.ones_like(z)
    conv = (conv_direct if direct else conv_fft)(one, z, one, h, mode)     # K conv z  (gates of the conv oracle = 1)
    gated = sigmoid(v) * conv                               # outer gate
    y = rms_norm(gated, g_out, eps)                         # RMSNorm before the residual addition
    return (y, gated) if parts else y
