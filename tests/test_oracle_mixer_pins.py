"""Pins of the Eq. 2 oracle (oracle/mixer.py): an independent scalar evaluation of a two-channel, two-token case,
a composition of library routines (torch fp64), closed forms and invariances.  None of them calls the CUDA path."""
import math

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import mixer

RNG = np.random.default_rng(20260719)


def rnd(*shape):
    return RNG.standard_normal(shape)


def test_scalar_evaluation_of_a_two_channel_causal_case():
    """B = 1, C = 2, L = 2, causal, eps = 0: every step of Eq. 2 evaluated with scalar arithmetic."""
    q = np.array([[[3.0, 0.0], [4.0, 1.0]]])            # [1, C=2, L=2]: token 0 = (3, 4), token 1 = (0, 1)
    k = np.array([[[1.0, -2.0], [0.5, 3.0]]])
    v = np.array([[[0.0, 1.0], [-1.0, 2.0]]])
    h = np.array([[[2.0, -1.0], [1.0, 0.5]]])           # causal taps K(0), K(1) per channel
    g_in, g_out = np.array([1.0, 2.0]), np.array([0.5, 1.0])
    sil = lambda x: x / (1.0 + math.exp(-x))
    sig = lambda x: 1.0 / (1.0 + math.exp(-x))
    # l2 over channels: token 0 has norm 5, token 1 norm 1
    a = [[3 / 5, 0.0], [4 / 5, 1.0]]                    # [c][t]
    inner = [[a[c][t] * sil(k[0, c, t]) for t in range(2)] for c in range(2)]
    z = [[0.0, 0.0], [0.0, 0.0]]
    for t in range(2):
        rms = math.sqrt((inner[0][t] ** 2 + inner[1][t] ** 2) / 2)
        for c in range(2):
            z[c][t] = inner[c][t] / rms * g_in[c]
    conv = [[h[0, c, 0] * z[c][0], h[0, c, 0] * z[c][1] + h[0, c, 1] * z[c][0]] for c in range(2)]
    gated = [[sig(v[0, c, t]) * conv[c][t] for t in range(2)] for c in range(2)]
    want = np.zeros((1, 2, 2))
    for t in range(2):
        rms = math.sqrt((gated[0][t] ** 2 + gated[1][t] ** 2) / 2)
        for c in range(2):
            want[0, c, t] = gated[c][t] / rms * g_out[c]
    for direct in (True, False):
        got = mixer.hyena_mixer(q, k, v, h, g_in, g_out, eps=0.0, mode="causal", direct=direct)
        np.testing.assert_allclose(got, want, rtol=1e-13, atol=1e-15)
    # token 1 of channel 0 has l2(q) = 0: its inner value is 0 whatever k is
    assert inner[0][1] == 0.0


@pytest.mark.parametrize("dims,mode", [((9,), "causal"), ((6, 5), "linear"), ((4, 3, 2), "linear"), ((8, 4), "circular")],
                         ids=str)
def test_against_a_composition_of_library_routines(dims, mode):
    """torch fp64: F.normalize, F.silu, F.rms_norm, torch.sigmoid and a direct convolution (conv{1,2,3}d with the
    flipped kernel; periodic padding for the circular mode)."""
    B, C, eps = 2, 3, 1e-5
    nd = len(dims)
    q, k, v = (torch.from_numpy(rnd(B, C, *dims)) for _ in range(3))
    taps = tuple(L if mode != "linear" else 2 * L - 1 for L in dims)
    h = torch.from_numpy(rnd(B, C, *taps))
    g_in, g_out = torch.from_numpy(rnd(C)), torch.from_numpy(rnd(C))
    perm = (0,) + tuple(range(2, 2 + nd)) + (1,)            # channels last for the normalisations
    inv = (0, nd + 1) + tuple(range(1, nd + 1))
    inner = F.normalize(q, p=2, dim=1, eps=1e-12) * F.silu(k)
    z = F.rms_norm(inner.permute(perm), (C,), g_in, eps).permute(inv)
    conv_fn = {1: F.conv1d, 2: F.conv2d, 3: F.conv3d}[nd]
    x = z.reshape(1, B * C, *dims)
    w = torch.flip(h.reshape(B * C, 1, *taps), dims=tuple(range(2, 2 + nd)))
    if mode == "linear":
        conv = conv_fn(x, w, padding=tuple(L - 1 for L in dims), groups=B * C)
    elif mode == "causal":
        conv = conv_fn(F.pad(x, (dims[0] - 1, 0)), w, groups=B * C)
    else:
        pad = []
        for L in reversed(dims):
            pad += [L - 1, 0]
        conv = conv_fn(F.pad(x, pad, mode="circular"), w, groups=B * C)
    conv = conv.reshape(B, C, *dims)
    want = F.rms_norm((torch.sigmoid(v) * conv).permute(perm), (C,), g_out, eps).permute(inv)
    got = mixer.hyena_mixer(q, k, v, h, g_in, g_out, eps=eps, mode=mode, direct=True)
    np.testing.assert_allclose(got, want.numpy(), rtol=1e-11, atol=1e-12)
    got2 = mixer.hyena_mixer(q, k, v, h, g_in, g_out, eps=eps, mode=mode, direct=False)
    np.testing.assert_allclose(got2, want.numpy(), rtol=1e-9, atol=1e-11)


def test_single_channel_closed_form():
    """C = 1, eps = 0, delta kernel: every normalisation reduces to a sign, so y = sign(q k) sign(g_in) g_out
    (SiLU keeps the sign of k, Sigmoid is positive)."""
    L = 16
    q, k, v = rnd(2, 1, L), rnd(2, 1, L), rnd(2, 1, L)
    h = np.zeros((1, 2 * L - 1))
    h[0, L - 1] = 1.7
    g_in, g_out = np.array([-0.3]), np.array([2.5])
    got = mixer.hyena_mixer(q, k, v, h, g_in, g_out, eps=0.0)
    np.testing.assert_allclose(got, np.sign(q * k) * -1.0 * 2.5, rtol=1e-12)


def test_invariances():
    dims, B, C = (7, 5), 2, 4
    q, k, v = rnd(B, C, *dims), rnd(B, C, *dims), rnd(B, C, *dims)
    h = rnd(B, C, 13, 9)
    g_in, g_out = rnd(C), rnd(C)
    base = mixer.hyena_mixer(q, k, v, h, g_in, g_out, eps=0.0)
    # l2(q) removes any positive per-token scale of q
    scale = np.exp(rnd(B, 1, *dims))
    np.testing.assert_allclose(mixer.hyena_mixer(q * scale, k, v, h, g_in, g_out, eps=0.0), base, rtol=1e-10, atol=1e-12)
    # with eps = 0 the last RMSNorm removes a global scale of the kernel and of g_in
    np.testing.assert_allclose(mixer.hyena_mixer(q, k, v, 3.0 * h, 0.25 * g_in, g_out, eps=0.0), base, rtol=1e-10, atol=1e-12)
    # linear in g_out; k = 0 silences the operator (eps > 0)
    np.testing.assert_allclose(mixer.hyena_mixer(q, k, v, h, g_in, -2.0 * g_out, eps=0.0), -2.0 * base, rtol=1e-12)
    assert np.all(mixer.hyena_mixer(q, 0 * k, v, h, g_in, g_out, eps=1e-6) == 0.0)
    # channels are exchangeable when their parameters move with them
    p = np.array([2, 0, 3, 1])
    moved = mixer.hyena_mixer(q[:, p], k[:, p], v[:, p], h[:, p], g_in[p], g_out[p], eps=0.0)
    np.testing.assert_allclose(moved, base[:, p], rtol=1e-10, atol=1e-12)
    # eps enters inside the roots: a huge eps scales the output down by about 1/eps (two roots)
    big = mixer.hyena_mixer(q, k, v, h, g_in, g_out, eps=1e12)
    assert np.max(np.abs(big)) < 1e-9
