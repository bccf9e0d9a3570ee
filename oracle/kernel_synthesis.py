"""CPU oracle of the input-dependent kernel K(x) of HyenaND -- TEST INFRASTRUCTURE ONLY.

    K(x)[b, c, i] = w_c(c_i) * f_theta(c_i; gamma_b, beta_b)[c]                    (Section 3.2.1, 3.2.2)

  f_theta    SIREN with J hidden layers of width H_f (Eq. 3), each hidden activation FiLM-modulated (Eq. 4):
                 a_1 = sin(omega_0 * (W_1 c_i + b_1)),      a_1 <- gamma_1 * a_1 + beta_1
                 a_j = sin(W_j a_{j-1} + b_j),              a_j <- gamma_j * a_j + beta_j      (j = 2..J)
                 f   = W_out a_J + b_out                    (C outputs, one per channel)
  w_c        Gaussian window exp(-1/2 sum_d (c_{i,d} / sigma_{d,c})^2) (Eq. 6), or, for causal 1-D kernels,
             the exponential window exp(-alpha_c |c_i|) with negative displacements removed (Appendix A.3)
  c_i        normalised coordinate of tap i on the kernel grid, per axis:
                 linear    displacement d in [-(L-1), L-1]  ->  d / (L-1)   (in [-1, 1]; 0 when L = 1)
                 causal    displacement t in [0, L-1]       ->  t / (L-1)
                 circular  tap m in [0, L): wrapped displacement d = m if m <= L/2 else m - L  ->  d / (L/2)
in plain numpy float64, one statement per step.  gamma, beta: [B, J, H_f] (the output of the FiLM network on the
control variable z(x); all ones / zeros give the static kernel).

Readings where the paper leaves a choice: Eq. 3 prints no biases (pass zeros for it; SIREN layers usually carry
them, so the oracle accepts them); FiLM acts on the activation after the sine; window and SIREN share the
normalised coordinates; the taps are laid out as the convolution expects them (oracle/__init__.py).
"""
from __future__ import annotations

import numpy as np


def axis_coordinates(L: int, mode: str) -> np.ndarray:
    """Normalised coordinate of every tap along one axis."""
    if mode == "linear":
        d = np.arange(-(L - 1), L, dtype=np.float64)
        return d / (L - 1) if L > 1 else np.zeros(1)
    if mode == "causal":
        t = np.arange(L, dtype=np.float64)
        return t / (L - 1) if L > 1 else np.zeros(1)
    if mode == "circular":
        m = np.arange(L, dtype=np.float64)
        d = np.where(m <= L / 2, m, m - L)
        return d / (L / 2) if L > 1 else np.zeros(1)
    raise ValueError(mode)


def coordinates(dims, mode: str) -> np.ndarray:
    """[K_1, .., K_N, N] array of tap coordinates."""
    axes = [axis_coordinates(L, mode) for L in dims]
    mesh = np.meshgrid(*axes, indexing="ij")
    return np.stack(mesh, axis=-1)


def synthesize(dims, mode, W1, b1, omega0, Wh, bh, Wout, bout, gamma, beta, window) -> np.ndarray:
    """K(x) as [B, C, K_1..K_N].
    W1 [H_f, N], b1 [H_f], omega0 [H_f]; Wh [J-1, H_f, H_f], bh [J-1, H_f]; Wout [C, H_f], bout [C];
    gamma, beta [B, J, H_f]; window: sigma [N, C] (Gaussian) or alpha [C] (causal exponential)."""
    W1, b1, omega0, Wh, bh, Wout, bout, gamma, beta, window = (
        np.asarray(a, dtype=np.float64) for a in (W1, b1, omega0, Wh, bh, Wout, bout, gamma, beta, window))
    dims = tuple(int(d) for d in dims)
    coords = coordinates(dims, mode)                      # [K.., N]
    taps = coords.shape[:-1]
    c = coords.reshape(-1, len(dims))                     # [T, N]
    B, J, Hf = gamma.shape
    C = Wout.shape[0]
    out = np.empty((B, C) + taps)
    if mode == "causal":
        win = np.exp(-window[None, :] * np.abs(c[:, :1]))                         # [T, C]; all displacements are >= 0 here
    else:
        win = np.exp(-0.5 * np.sum((c[:, :, None] / window[None, :, :]) ** 2, axis=1))   # [T, C]
    for b in range(B):
        a = np.sin(omega0[None, :] * (c @ W1.T + b1[None, :]))
        a = gamma[b, 0][None, :] * a + beta[b, 0][None, :]
        for j in range(1, J):
            a = np.sin(a @ Wh[j - 1].T + bh[j - 1][None, :])
            a = gamma[b, j][None, :] * a + beta[b, j][None, :]
        f = a @ Wout.T + bout[None, :]                    # [T, C]
        out[b] = (win * f).T.reshape((C,) + taps)
    return out
