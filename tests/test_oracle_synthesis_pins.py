"""Pins of the kernel-synthesis oracle (oracle/kernel_synthesis.py): coordinates and window values worked by hand,
closed forms of degenerate networks, a torch fp64 composition, FiLM identities.  None of them calls the CUDA path."""
import math

import numpy as np
import pytest
import torch

from oracle import kernel_synthesis as ks

RNG = np.random.default_rng(31)


def params(N, Hf, J, C, B):
    return dict(W1=RNG.standard_normal((Hf, N)), b1=RNG.standard_normal(Hf), omega0=RNG.uniform(1, 30, Hf),
                Wh=RNG.standard_normal((J - 1, Hf, Hf)) / math.sqrt(Hf), bh=RNG.standard_normal((J - 1, Hf)),
                Wout=RNG.standard_normal((C, Hf)) / math.sqrt(Hf), bout=RNG.standard_normal(C),
                gamma=1 + 0.3 * RNG.standard_normal((B, J, Hf)), beta=0.3 * RNG.standard_normal((B, J, Hf)))


def test_coordinates_by_hand():
    np.testing.assert_allclose(ks.axis_coordinates(3, "linear"), [-1, -0.5, 0, 0.5, 1])
    np.testing.assert_allclose(ks.axis_coordinates(5, "causal"), [0, 0.25, 0.5, 0.75, 1])
    # 8 taps on a ring: displacements 0 1 2 3 4 -3 -2 -1, half the ring = 4
    np.testing.assert_allclose(ks.axis_coordinates(8, "circular"), [0, 0.25, 0.5, 0.75, 1, -0.75, -0.5, -0.25])
    np.testing.assert_allclose(ks.axis_coordinates(1, "linear"), [0])
    c = ks.coordinates((2, 3), "linear")
    assert c.shape == (3, 5, 2)
    np.testing.assert_allclose(c[0, 4], [-1, 1])          # displacement (-1, +2) of a 2 x 3 grid
    np.testing.assert_allclose(c[1, 2], [0, 0])           # the centre tap is displacement zero


def test_zero_network_returns_window_times_bias():
    """All weights zero: f = b_out, so K = w * b_out; the Gaussian window by hand at three taps."""
    dims, C, Hf, J = (3, 2), 2, 4, 2
    p = params(2, Hf, J, C, 1)
    p["W1"][:] = 0; p["b1"][:] = 0; p["Wh"][:] = 0; p["bh"][:] = 0; p["Wout"][:] = 0
    p["bout"] = np.array([2.0, -3.0])
    sigma = np.array([[0.5, 1.0], [2.0, 0.25]])           # [axis, channel]
    K = ks.synthesize(dims, "linear", window=sigma, **p)
    assert K.shape == (1, 2, 5, 3)
    # centre tap: window 1
    np.testing.assert_allclose(K[0, :, 2, 1], [2.0, -3.0])
    # tap (0, 0): displacement (-2, -1) -> coordinates (-1, -1)
    np.testing.assert_allclose(K[0, 0, 0, 0], 2.0 * math.exp(-0.5 * ((1 / 0.5) ** 2 + (1 / 2.0) ** 2)))
    np.testing.assert_allclose(K[0, 1, 0, 0], -3.0 * math.exp(-0.5 * ((1 / 1.0) ** 2 + (1 / 0.25) ** 2)))
    # tap (3, 2): displacement (+1, +1) -> coordinates (0.5, 1)
    np.testing.assert_allclose(K[0, 0, 3, 2], 2.0 * math.exp(-0.5 * ((0.5 / 0.5) ** 2 + (1 / 2.0) ** 2)))


def test_one_unit_network_closed_form_and_causal_window():
    """J = 1, H_f = 1, C = 1: K(t) = exp(-alpha c) * (w_out (gamma sin(omega (w c + b)) + beta) + b_out), c = t/(L-1)."""
    L = 9
    w, b, om, wo, bo, ga, be, al = 0.7, -0.2, 11.0, 1.5, 0.1, 1.3, -0.4, 2.5
    K = ks.synthesize((L,), "causal", W1=[[w]], b1=[b], omega0=[om], Wh=np.zeros((0, 1, 1)), bh=np.zeros((0, 1)),
                      Wout=[[wo]], bout=[bo], gamma=[[[ga]]], beta=[[[be]]], window=[al])
    want = [math.exp(-al * t / (L - 1)) * (wo * (ga * math.sin(om * (w * t / (L - 1) + b)) + be) + bo) for t in range(L)]
    np.testing.assert_allclose(K[0, 0], want, rtol=1e-13)


@pytest.mark.parametrize("dims,mode", [((7,), "causal"), ((5, 4), "linear"), ((3, 4, 2), "linear"), ((8, 4), "circular")],
                         ids=str)
def test_against_a_torch_composition(dims, mode):
    N, Hf, J, C, B = len(dims), 6, 3, 4, 2
    p = params(N, Hf, J, C, B)
    window = RNG.uniform(0.5, 3.0, C) if mode == "causal" else RNG.uniform(0.2, 1.5, (N, C))
    got = ks.synthesize(dims, mode, window=window, **p)
    t = {k: torch.from_numpy(np.asarray(v)) for k, v in p.items()}
    coords = torch.from_numpy(ks.coordinates(dims, mode))
    lin = torch.nn.functional.linear
    for b in range(B):
        a = torch.sin(t["omega0"] * lin(coords, t["W1"], t["b1"]))
        a = t["gamma"][b, 0] * a + t["beta"][b, 0]
        for j in range(1, J):
            a = torch.sin(lin(a, t["Wh"][j - 1], t["bh"][j - 1]))
            a = t["gamma"][b, j] * a + t["beta"][b, j]
        f = lin(a, t["Wout"], t["bout"])                  # [K.., C]
        if mode == "causal":
            win = torch.exp(-torch.from_numpy(window) * coords[..., :1].abs())
        else:
            win = torch.exp(-0.5 * ((coords[..., None] / torch.from_numpy(window)) ** 2).sum(dim=-2))
        want = torch.movedim(win * f, -1, 0)
        np.testing.assert_allclose(got[b], want.numpy(), rtol=1e-11, atol=1e-13)


def test_film_identities():
    dims, N, Hf, J, C = (6, 5), 2, 5, 2, 3
    p = params(N, Hf, J, C, 2)
    sigma = RNG.uniform(0.3, 1.0, (N, C))
    p["gamma"][1] = 1.0
    p["beta"][1] = 0.0
    K = ks.synthesize(dims, "linear", window=sigma, **p)
    # identity modulation (gamma = 1, beta = 0) is the static kernel: the same for any batch entry that has it
    q = dict(p, gamma=np.ones((1, J, Hf)), beta=np.zeros((1, J, Hf)))
    np.testing.assert_allclose(K[1], ks.synthesize(dims, "linear", window=sigma, **q)[0], rtol=1e-14)
    assert np.max(np.abs(K[0] - K[1])) > 1e-3
    # modulation of the last hidden layer is affine in the output: K(gamma_J, beta_J) - K(gamma_J, 0) = w * W_out beta_J
    r = dict(p)
    r["beta"] = p["beta"].copy()
    r["beta"][0, J - 1] = 0.0
    diff = K[0] - ks.synthesize(dims, "linear", window=sigma, **r)[0]
    shift = p["Wout"] @ p["beta"][0, J - 1]
    c = ks.coordinates(dims, "linear")
    win = np.exp(-0.5 * np.sum((c[..., None] / sigma) ** 2, axis=-2))
    np.testing.assert_allclose(diff, np.moveaxis(win * shift, -1, 0), rtol=1e-10, atol=1e-13)
    # the Gaussian window is even and the centre tap has weight one
    s = dict(q, W1=np.zeros((Hf, N)))                      # a network that ignores the coordinate
    Ks = ks.synthesize(dims, "linear", window=sigma, **s)[0]
    np.testing.assert_allclose(Ks, Ks[:, ::-1, ::-1], rtol=1e-13)
