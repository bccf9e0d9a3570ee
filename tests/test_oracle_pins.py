"""Pins for the CPU oracle: everything here checks oracle/ against facts that do
not come from the oracle itself -- hand-worked examples of the definition,
closed forms, invariants, library routines used as black boxes, brute force.
No GPU, no CUDA library."""
import itertools
import json
import os

import numpy as np
import pytest
import scipy.signal
import torch

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "worked_examples.json")
RNG = np.random.default_rng(1234)


def rnd(*shape):
    return RNG.standard_normal(shape)


def both(q, k, v, h, mode="linear"):
    """O1 and O2 must agree (convolution theorem); returns O1."""
    a = oracle.conv_direct(q, k, v, h, mode)
    b = oracle.conv_fft(q, k, v, h, mode)
    assert oracle.rel_l2(b, a) < 1e-12
    return a


# ---- worked examples (hand expansion of Definition A.2/A.3) -------------------

def _golden_cases():
    with open(GOLDEN) as f:
        return json.load(f)["cases"]


@pytest.mark.parametrize("case", _golden_cases(), ids=lambda c: c["name"])
def test_worked_examples(case):
    dims = case["dims"]
    u = np.array(case["u"], dtype=float).reshape([1, 1] + dims)
    q = np.array(case["q"], dtype=float).reshape([1, 1] + dims)
    if "h" in case:
        h = np.array(case["h"], dtype=float).reshape(1, 1, -1)
    else:
        taps = [2 * L - 1 for L in dims]
        h = np.zeros([1, 1] + taps)
        for key, val in case["h_nonzero"].items():
            d = [int(t) for t in key.split(",")]
            h[(0, 0) + tuple(di + L - 1 for di, L in zip(d, dims))] = val
    ones = np.ones_like(u)
    for fn in (oracle.conv_direct, oracle.conv_fft):
        conv = fn(ones, u, ones, h, case["mode"])
        y = fn(q, u, ones, h, case["mode"])
        np.testing.assert_allclose(conv.reshape(dims), np.array(case["conv"], float), atol=1e-12)
        np.testing.assert_allclose(y.reshape(dims), np.array(case["y"], float), atol=1e-12)
        # the gate factors commute: k=1, v=u gives the same result
        y2 = fn(q, ones, u, h, case["mode"])
        np.testing.assert_allclose(y2, y, atol=1e-12)


# ---- delta / impulse: orientation, centre tap, no wrap-around -----------------

SHAPES = [(1,), (2,), (3,), (5,), (15, 14), (3, 5), (5, 3, 2), (7, 1, 4), (8, 8)]


@pytest.mark.parametrize("dims", SHAPES)
def test_delta_filter_returns_gated_input(dims):
    B, C = 2, 3
    q, k, v = rnd(B, C, *dims), rnd(B, C, *dims), rnd(B, C, *dims)
    taps = tuple(2 * L - 1 for L in dims)
    h = np.zeros((B, C) + taps)
    s = rnd(C)
    h[(slice(None), slice(None)) + tuple(L - 1 for L in dims)] = s[None, :]
    y = both(q, k, v, h)
    np.testing.assert_allclose(y, s.reshape(1, C, *[1] * len(dims)) * q * k * v, atol=1e-12)


def test_shifted_delta_no_wraparound():
    dims = (3, 5, 2)
    B, C = 1, 2
    q, k, v = rnd(B, C, *dims), rnd(B, C, *dims), rnd(B, C, *dims)
    u = k * v
    for d in [(1, 0, 0), (0, -2, 0), (0, 0, 1), (-2, 4, -1), (2, -4, 1)]:
        h = np.zeros((B, C) + tuple(2 * L - 1 for L in dims))
        h[(slice(None), slice(None)) + tuple(di + L - 1 for di, L in zip(d, dims))] = 1.0
        y = both(q, k, v, h)
        exp = np.zeros_like(u)
        for i in itertools.product(*[range(L) for L in dims]):
            j = tuple(ii - di for ii, di in zip(i, d))
            if all(0 <= jj < L for jj, L in zip(j, dims)):
                exp[(slice(None), slice(None)) + i] = u[(slice(None), slice(None)) + j]
        np.testing.assert_allclose(y, q * exp, atol=1e-12)


def test_unit_impulse_reads_filter_back():
    dims = (3, 5, 2)
    taps = tuple(2 * L - 1 for L in dims)
    h = rnd(1, 1, *taps)
    ones = np.ones((1, 1) + dims)
    for j0 in [(0, 0, 0), (2, 4, 1), (1, 2, 0)]:
        u = np.zeros((1, 1) + dims)
        u[(0, 0) + j0] = 1.0
        y = both(ones, u, ones, h)
        for i in itertools.product(*[range(L) for L in dims]):
            tap = tuple(ii - jj + L - 1 for ii, jj, L in zip(i, j0, dims))
            assert abs(y[(0, 0) + i] - h[(0, 0) + tap]) < 1e-12


# ---- library routines as black boxes ------------------------------------------

@pytest.mark.parametrize("dims", [(5,), (16,), (3, 5), (15, 14), (5, 3, 2), (6, 7, 4)])
def test_against_scipy_full_convolution(dims):
    B, C = 2, 2
    q, k, v = rnd(B, C, *dims), rnd(B, C, *dims), rnd(B, C, *dims)
    h = rnd(B, C, *[2 * L - 1 for L in dims])
    y = both(q, k, v, h)
    crop = tuple(slice(L - 1, 2 * L - 1) for L in dims)
    for b in range(B):
        for c in range(C):
            full = scipy.signal.convolve(k[b, c] * v[b, c], h[b, c], mode="full", method="direct")
            np.testing.assert_allclose(y[b, c], q[b, c] * full[crop], atol=1e-11)


@pytest.mark.parametrize("L", [1, 2, 7, 33])
def test_causal_against_numpy_convolve(L):
    B, C = 2, 3
    q, k, v = rnd(B, C, L), rnd(B, C, L), rnd(B, C, L)
    h = rnd(C, L)                                     # shared over the batch
    y = both(q, k, v, h, "causal")
    for b in range(B):
        for c in range(C):
            np.testing.assert_allclose(y[b, c], q[b, c] * np.convolve(k[b, c] * v[b, c], h[c])[:L],
                                       atol=1e-12)


@pytest.mark.parametrize("dims", [(9,), (6, 5), (4, 3, 5)])
def test_against_torch_conv_fp64(dims):
    B, C = 2, 3
    q, k, v = rnd(B, C, *dims), rnd(B, C, *dims), rnd(B, C, *dims)
    h = rnd(B, C, *[2 * L - 1 for L in dims])
    y = both(q, k, v, h)
    conv = {1: torch.nn.functional.conv1d, 2: torch.nn.functional.conv2d,
            3: torch.nn.functional.conv3d}[len(dims)]
    axes = tuple(range(2, 2 + len(dims)))
    for b in range(B):
        x = torch.from_numpy(k[b] * v[b])[None]                      # [1, C, ...]
        w = torch.from_numpy(np.flip(h[b], axis=tuple(a - 1 for a in axes)).copy())[:, None]
        out = conv(x, w, padding=[L - 1 for L in dims], groups=C)[0].numpy()
        np.testing.assert_allclose(y[b], q[b] * out, atol=1e-11)


def test_fftn_against_numpy_and_parseval():
    for shape in [(8,), (4, 16), (2, 8, 4), (1, 32)]:
        x = rnd(*shape) + 1j * rnd(*shape)
        X = oracle.fftn(x)
        np.testing.assert_allclose(X, np.fft.fftn(x), atol=1e-11)
        np.testing.assert_allclose(oracle.fftn(X, inverse=True) / x.size, x, atol=1e-12)
        assert abs(np.sum(np.abs(x) ** 2) - np.sum(np.abs(X) ** 2) / x.size) < 1e-9


def test_parseval_of_circular_convolution():
    dims = (8, 4)
    k, v, h = rnd(1, 1, *dims), rnd(1, 1, *dims), rnd(1, 1, *dims)
    ones = np.ones((1, 1) + dims)
    w = both(ones, k, v, h, "circular")[0, 0]
    U, H = np.fft.fftn(k[0, 0] * v[0, 0]), np.fft.fftn(h[0, 0])
    assert abs(np.sum(w ** 2) - np.sum(np.abs(U) ** 2 * np.abs(H) ** 2) / w.size) < 1e-9


# ---- Toeplitz / separable-attention form (Theorem A.5) -------------------------

def test_dense_toeplitz_form_1d():
    L = 17
    q, k, v = rnd(1, 1, L), rnd(1, 1, L), rnd(1, 1, L)
    h = rnd(1, 1, 2 * L - 1)
    T = np.array([[h[0, 0, i - j + L - 1] for j in range(L)] for i in range(L)])
    A = np.diag(q[0, 0]) @ T @ np.diag(k[0, 0] * v[0, 0])        # A = D_l T D_R
    y = both(q, k, v, h)
    np.testing.assert_allclose(y[0, 0], A @ np.ones(L), atol=1e-12)
    hc = rnd(1, 1, L)
    Tc = np.array([[hc[0, 0, i - j] if i >= j else 0.0 for j in range(L)] for i in range(L)])
    yc = both(q, k, v, hc, "causal")
    np.testing.assert_allclose(yc[0, 0], np.diag(q[0, 0]) @ Tc @ (k[0, 0] * v[0, 0]), atol=1e-12)


def test_block_toeplitz_form_2d():
    L1, L2 = 4, 5
    q, k, v = rnd(1, 1, L1, L2), rnd(1, 1, L1, L2), rnd(1, 1, L1, L2)
    h = rnd(1, 1, 2 * L1 - 1, 2 * L2 - 1)
    n = L1 * L2
    T = np.zeros((n, n))
    for i1, i2, j1, j2 in itertools.product(range(L1), range(L2), range(L1), range(L2)):
        T[i1 * L2 + i2, j1 * L2 + j2] = h[0, 0, i1 - j1 + L1 - 1, i2 - j2 + L2 - 1]
    y = both(q, k, v, h)
    np.testing.assert_allclose(y[0, 0].ravel(), q.ravel() * (T @ (k * v).ravel()), atol=1e-12)


# ---- closed forms and invariants -------------------------------------------------

def test_all_ones_filter_closed_forms():
    L = 11
    q, k, v = rnd(2, 2, L), rnd(2, 2, L), rnd(2, 2, L)
    yc = both(q, k, v, np.ones((2, L)), "causal")
    np.testing.assert_allclose(yc, q * np.cumsum(k * v, axis=-1), atol=1e-12)
    dims = (4, 3, 2)
    q, k, v = rnd(1, 2, *dims), rnd(1, 2, *dims), rnd(1, 2, *dims)
    y = both(q, k, v, np.ones((1, 2, 7, 5, 3)))
    np.testing.assert_allclose(y, q * (k * v).sum(axis=(2, 3, 4), keepdims=True), atol=1e-12)


def test_linearity_in_each_argument():
    dims = (6, 5)
    B, C = 2, 2
    q, k, v, h = rnd(B, C, *dims), rnd(B, C, *dims), rnd(B, C, *dims), rnd(B, C, 11, 9)
    q2, k2, v2, h2 = rnd(B, C, *dims), rnd(B, C, *dims), rnd(B, C, *dims), rnd(B, C, 11, 9)
    a, b = 0.7, -1.3
    f = oracle.conv_direct
    np.testing.assert_allclose(f(q, k, v, a * h + b * h2), a * f(q, k, v, h) + b * f(q, k, v, h2), atol=1e-11)
    np.testing.assert_allclose(f(a * q + b * q2, k, v, h), a * f(q, k, v, h) + b * f(q2, k, v, h), atol=1e-11)
    np.testing.assert_allclose(f(q, a * k + b * k2, v, h), a * f(q, k, v, h) + b * f(q, k2, v, h), atol=1e-11)
    np.testing.assert_allclose(f(q, k, a * v + b * v2, h), a * f(q, k, v, h) + b * f(q, k, v2, h), atol=1e-11)


def test_circular_shift_equivariance_and_numpy_circular():
    dims = (8, 4)
    k, v, h = rnd(1, 2, *dims), np.ones((1, 2) + dims), rnd(1, 2, *dims)
    ones = np.ones((1, 2) + dims)
    base = both(ones, k, v, h, "circular")
    for d in [(1, 0), (0, 3), (5, 2)]:
        moved = both(ones, np.roll(k, d, axis=(2, 3)), v, h, "circular")
        np.testing.assert_allclose(moved, np.roll(base, d, axis=(2, 3)), atol=1e-12)
    ref = np.fft.ifftn(np.fft.fftn(k, axes=(2, 3)) * np.fft.fftn(h, axes=(2, 3)), axes=(2, 3)).real
    np.testing.assert_allclose(base, ref, atol=1e-12)


def test_linear_shift_equivariance_inside_the_grid():
    L = 16
    u = np.zeros((1, 1, L))
    u[0, 0, 2:6] = rnd(4)
    h = np.zeros((1, 1, 2 * L - 1))
    h[0, 0, L - 1 - 2:L - 1 + 3] = rnd(5)             # displacements -2..2
    ones = np.ones((1, 1, L))
    a = both(ones, u, ones, h)
    b = both(ones, np.roll(u, 5, axis=-1), ones, h)
    np.testing.assert_allclose(b, np.roll(a, 5, axis=-1), atol=1e-12)


def test_separable_filter_is_successive_1d_convolutions():
    dims = (5, 4, 3)
    u = rnd(*dims)
    h1, h2, h3 = rnd(9), rnd(7), rnd(5)
    h = np.einsum("a,b,c->abc", h1, h2, h3)[None, None]
    ones = np.ones((1, 1) + dims)
    y = both(ones, u[None, None], ones, h)[0, 0]
    step = u
    for ax, (hk, L) in enumerate(zip((h1, h2, h3), dims)):
        step = np.apply_along_axis(lambda r: np.convolve(r, hk)[L - 1:2 * L - 1], ax, step)
    np.testing.assert_allclose(y, step, atol=1e-12)


def test_shortcut_term_equals_centre_tap():
    """y = K*x + s.x (Definition A.2) is the same as adding s to the zero-displacement tap."""
    L = 9
    q, k, v, h = rnd(1, 2, L), rnd(1, 2, L), rnd(1, 2, L), rnd(1, 2, 2 * L - 1)
    s = rnd(2)
    h2 = h.copy()
    h2[0, :, L - 1] += s
    np.testing.assert_allclose(both(q, k, v, h2), both(q, k, v, h) + q * s[None, :, None] * k * v, atol=1e-12)


def test_causality_is_bit_exact_in_o1():
    L = 12
    q, k, v, h = rnd(1, 1, L), rnd(1, 1, L), rnd(1, 1, L), rnd(1, L)
    base = oracle.conv_direct(q, k, v, h, "causal")
    for t in (0, 3, 7):
        k2, v2 = k.copy(), v.copy()
        k2[..., t + 1:] = rnd(L - t - 1)
        v2[..., t + 1:] = rnd(L - t - 1)
        other = oracle.conv_direct(q, k2, v2, h, "causal")
        assert np.array_equal(other[..., :t + 1], base[..., :t + 1])


def test_direct_at_matches_whole_tensor_and_shared_filter():
    dims = (6, 5)
    B, C = 3, 2
    q, k, v = rnd(B, C, *dims), rnd(B, C, *dims), rnd(B, C, *dims)
    h = rnd(C, 11, 9)
    full = both(q, k, v, h)
    tiled = both(q, k, v, np.broadcast_to(h, (B,) + h.shape).copy())
    np.testing.assert_allclose(full, tiled, atol=0)
    idx = RNG.integers(0, full.size, size=40)
    np.testing.assert_allclose(oracle.conv_direct_at(q, k, v, h, idx), full.ravel()[idx], atol=0)


def test_bf16_inputs_are_widened_exactly():
    dims = (5, 4)
    q = torch.randn(1, 2, *dims).bfloat16()
    k = torch.randn(1, 2, *dims).bfloat16()
    v = torch.randn(1, 2, *dims).bfloat16()
    h = torch.randn(1, 2, 9, 7).bfloat16()
    a = oracle.conv_direct(q, k, v, h)
    b = oracle.conv_direct(q.double().numpy(), k.double().numpy(), v.double().numpy(), h.double().numpy())
    assert np.array_equal(a, b)


def test_argument_errors():
    with pytest.raises(ValueError):
        oracle.conv_direct(rnd(1, 1, 4), rnd(1, 1, 4), rnd(1, 1, 4), rnd(1, 1, 6))
    with pytest.raises(ValueError):
        oracle.conv_direct(rnd(1, 1, 4, 4), rnd(1, 1, 4, 4), rnd(1, 1, 4, 4), rnd(1, 1, 4, 4), "causal")


LARGE_PADDED = [((32768,), "linear"), ((32768,), "causal"), ((128, 128), "linear"), ((32, 64, 64), "linear")]


@pytest.mark.parametrize("dims,mode", LARGE_PADDED, ids=str)
def test_o2_agrees_with_sampled_o1_at_large_padded_sizes(dims, mode):
    """Convolution theorem at the sizes the GPU tests rely on O2 for (padded 2^16, 256 x 256, 64 x 128 x 128):
    the FFT path against the defining sum evaluated at seeded output positions, per-sample and shared filters."""
    rng = np.random.default_rng(7)
    B, C = 2, 2
    taps = tuple(L if mode == "causal" else 2 * L - 1 for L in dims)
    q, k, v = (rng.standard_normal((B, C) + dims) for _ in range(3))
    for shared in (False, True):
        h = rng.standard_normal(((C,) if shared else (B, C)) + taps)
        full = oracle.conv_fft(q, k, v, h, mode)
        idx = rng.integers(0, full.size, size=96)
        at = oracle.conv_direct_at(q, k, v, h, idx, mode)
        scale = np.sqrt(np.mean(full * full))
        assert np.max(np.abs(full.ravel()[idx] - at)) <= 1e-11 * scale
