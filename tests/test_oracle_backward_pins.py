"""Pins of the backward oracle (oracle/backward.py).  The forward is multilinear (linear in each of q, k, v, h), so
<dy, forward(.., x + d, ..) - forward(.., x, ..)> = <dx, d> holds EXACTLY for any direction d: the gradients are pinned
to the already pinned forward oracle without any step size.  A second, independent pin is torch autograd through a
torch fp64 convolution; a third, a hand-worked 1-D case."""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

import oracle
from oracle import backward as ob

RNG = np.random.default_rng(5)
CASES = [((6,), "linear", False), ((7,), "causal", False), ((7,), "causal", True), ((8,), "circular", False),
         ((4, 5), "linear", True), ((4, 8), "circular", True), ((3, 2, 4), "linear", False)]


def make(dims, mode, shared, B=2, C=3):
    taps = tuple(2 * L - 1 if mode == "linear" else L for L in dims)
    q, k, v, dy = (RNG.standard_normal((B, C) + dims) for _ in range(4))
    h = RNG.standard_normal(((C,) if shared else (B, C)) + taps)
    return q, k, v, h, dy


def test_hand_worked_causal_case():
    """L = 3, causal, one channel: u = (1, 2, 3), h = (K0, K1, K2) = (2, -1, 0.5), q = (1, 2, -1), dy = (1, 1, 2).
    w = (2, 3, 4.5); g = dy q = (1, 2, -2).  du_j = sum_{i>=j} K(i-j) g_i: du_0 = 2*1 - 1*2 + 0.5*(-2) = -1,
    du_1 = 2*2 - 1*(-2) = 6, du_2 = 2*(-2) = -4.  dh_t = sum_i g_i u_{i-t}: dh_0 = 1*1 + 2*2 - 2*3 = -1,
    dh_1 = 2*1 - 2*2 = -2, dh_2 = -2*1 = -2."""
    k = np.array([[[1.0, 2.0, 3.0]]]); v = np.ones((1, 1, 3))
    h = np.array([[[2.0, -1.0, 0.5]]]); q = np.array([[[1.0, 2.0, -1.0]]]); dy = np.array([[[1.0, 1.0, 2.0]]])
    for direct in (True, False):
        dq, dk, dv, dh = ob.backward(q, k, v, h, dy, "causal", direct=direct)
        np.testing.assert_allclose(dq[0, 0], [2.0, 3.0, 9.0], atol=1e-12)
        np.testing.assert_allclose(dk[0, 0], [-1.0, 6.0, -4.0], atol=1e-12)
        np.testing.assert_allclose(dv[0, 0], [-1.0, 12.0, -12.0], atol=1e-12)
        np.testing.assert_allclose(dh[0, 0], [-1.0, -2.0, -2.0], atol=1e-12)


@pytest.mark.parametrize("dims,mode,shared", CASES, ids=str)
def test_exact_directional_derivatives_of_the_forward_oracle(dims, mode, shared):
    q, k, v, h, dy = make(dims, mode, shared)
    base = oracle.conv_direct(q, k, v, h, mode)
    for direct in (True, False):
        grads = ob.backward(q, k, v, h, dy, mode, direct=direct)
        for which, (x, gx) in enumerate(zip((q, k, v, h), grads)):
            d = RNG.standard_normal(x.shape)
            args = [q, k, v, h]
            args[which] = x + d
            lhs = np.sum(dy * (oracle.conv_direct(*args, mode) - base))
            rhs = np.sum(gx * d)
            assert abs(lhs - rhs) <= 1e-10 * max(1.0, abs(lhs)), (which, lhs, rhs)


@pytest.mark.parametrize("dims,mode,shared", CASES, ids=str)
def test_against_torch_autograd(dims, mode, shared):
    q, k, v, h, dy = make(dims, mode, shared)
    B, C = q.shape[:2]
    nd = len(dims)
    tq, tk, tv, th = (torch.from_numpy(a).requires_grad_(True) for a in (q, k, v, h))
    taps = th.shape[-nd:]
    hfull = th if not shared else th.unsqueeze(0).expand((B,) + th.shape)
    x = (tk * tv).reshape(1, B * C, *dims)
    wgt = torch.flip(hfull.reshape(B * C, 1, *taps), dims=tuple(range(2, 2 + nd)))
    conv_fn = {1: F.conv1d, 2: F.conv2d, 3: F.conv3d}[nd]
    if mode == "linear":
        w = conv_fn(x, wgt, padding=tuple(L - 1 for L in dims), groups=B * C)
    elif mode == "causal":
        w = conv_fn(F.pad(x, (dims[0] - 1, 0)), wgt, groups=B * C)
    else:
        pad = []
        for L in reversed(dims):
            pad += [L - 1, 0]
        w = conv_fn(F.pad(x, pad, mode="circular"), wgt, groups=B * C)
    y = tq * w.reshape(B, C, *dims)
    y.backward(torch.from_numpy(dy))
    got = ob.backward(q, k, v, h, dy, mode, direct=True)
    for a, t in zip(got, (tq, tk, tv, th)):
        np.testing.assert_allclose(a, t.grad.numpy(), rtol=1e-10, atol=1e-11)


def test_fft_correlation_agrees_with_the_definition_at_a_larger_size():
    q, k, v, h, dy = make((40, 33), "linear", False, B=1, C=2)
    a = ob.backward(q, k, v, h, dy, "linear", direct=True)
    b = ob.backward(q, k, v, h, dy, "linear", direct=False)
    for x, y in zip(a, b):
        np.testing.assert_allclose(x, y, rtol=1e-9, atol=1e-10)
