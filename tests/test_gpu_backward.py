"""GPU parity of the backward pass (hyenand_backward through the C ABI) against oracle/backward.py.

Each of dq, dk, dv, dh carries the gates of the forward: whole-tensor rel-L2 against the unrounded fp64 oracle
<= 1e-5 (fp32 I/O), <= 2e-3 and 1.1 x the output rounding (bf16 I/O), plus an element-wise bound: output rounding
plus the fp32 transform error relative to the rms level of the convolution result the element comes from."""
import numpy as np
import pytest
import torch

import oracle
from oracle import backward as ob
from paper_2607_19378_b200 import workloads as W
from parity_util import ELEM_C, ELEM_R, TOL

pytestmark = pytest.mark.gpu


def guarded(like):
    n = like.numel()
    big = torch.full((n + 512,), 7.0, dtype=like.dtype, device="cuda")
    t = big[256:256 + n].view(like.shape)
    t.fill_(float("nan"))
    return big, t


def run_backward(w, q, k, v, h, dy):
    from paper_2607_19378_b200 import hyenand as hn
    bw = hn.Backward(w.dims, w.B, w.C, mode=w.mode, dtype=w.torch_dtype)
    try:
        dq_, dk_, dv_, dh_, ddy = (t.cuda() for t in (q, k, v, h, dy))
        outs = [guarded(dq_), guarded(dq_), guarded(dq_), guarded(dh_)]
        stride = 0 if w.h_shared else w.C * h[0, 0].numel()
        for _ in range(2):                                  # twice: the scratch keeps nothing that must be cleared
            hn.hyenand_backward(bw.handle, dq_, dk_, dv_, dh_, stride, ddy, *[t for _, t in outs])
        torch.cuda.synchronize()
        assert hn.hyenand_backward_guard_damage(bw.handle) == 0
        for big, t in outs:
            assert bool((big[:256] == 7.0).all()) and bool((big[256 + t.numel():] == 7.0).all()), "a kernel wrote outside a gradient"
        return [t.cpu().clone() for _, t in outs]
    finally:
        bw.close()


def gate(name, got, ref, dtype, scale_level):
    err = oracle.rel_l2(got, ref)
    tol = TOL[dtype]
    if dtype == "bf16":
        rounding = oracle.rel_l2(torch.from_numpy(ref).bfloat16(), ref)
        assert err <= 1.1 * rounding + 1e-6, f"{name}: rel-L2 {err:.3e} vs rounding {rounding:.3e}"
        if ref.size < 4096:
            tol = max(tol, 1.1 * rounding)
    assert np.isfinite(err) and err <= tol, f"{name}: rel-L2 {err:.3e}"
    bound = ELEM_R[dtype] * np.abs(ref) + 2 * ELEM_C * scale_level + 1e-37
    ex = float(np.max(np.abs(oracle.to_f64(got) - ref) / bound))
    assert ex <= 1.0, f"{name}: an element is off by {ex:.2f} x its bound"


def check_backward(w, q, k, v, h, seed, direct=False):
    g = torch.Generator().manual_seed(seed)
    dy = torch.randn(q.shape, generator=g).to(q.dtype)
    got = run_backward(w, q, k, v, h, dy)
    ref = ob.backward(q, k, v, h, dy, w.mode, direct=direct)
    qd, kd, vd, dyd = (oracle.to_f64(t) for t in (q, k, v, dy))
    nd = len(w.dims)
    ax = tuple(range(2, 2 + nd))
    rms = lambda x: np.sqrt(np.mean(x * x, axis=ax, keepdims=True))
    conv_w = ref[0] / np.where(dyd != 0, dyd, 1.0)           # w = dq / dy
    du = ref[1] / np.where(vd != 0, vd, 1.0)
    gate("dq", got[0], ref[0], w.dtype, np.abs(dyd) * rms(conv_w))
    gate("dk", got[1], ref[1], w.dtype, np.abs(vd) * rms(du))
    gate("dv", got[2], ref[2], w.dtype, np.abs(kd) * rms(du))
    # dh: a correlation of g = dy q with u = k v; its transform error is relative to sqrt(sum g^2 sum u^2) / sqrt(taps) per slice
    gg, uu = dyd * qd, kd * vd
    lvl = np.sqrt(np.sum(gg * gg, axis=ax) * np.sum(uu * uu, axis=ax) / np.prod(w.dims))       # [B, C]
    if w.h_shared:
        lvl = np.sqrt(np.sum(lvl * lvl, axis=0))
    lvl = lvl.reshape(lvl.shape + (1,) * nd)
    gate("dh", got[3], ref[3], w.dtype, lvl)


SHAPES = [((1,), False), ((5,), False), ((300,), False), ((1000,), True), ((4096,), True), ((5000,), False),
          ((9001,), True), ((15, 14), False), ((40, 50), False), ((64, 64), False), ((130, 70), False),
          ((5, 3, 2), False), ((20, 24, 30), False), ((32, 32, 32), False), ((8, 40, 48), False), ((6, 36, 43), False)]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("shared", [False, True])
@pytest.mark.parametrize("dims,causal", SHAPES, ids=str)
def test_backward_matches_the_oracle(dims, causal, shared, dtype):
    w, (q, k, v, h) = W.random_problem(dims, B=2, C=3, dtype=dtype, causal=causal, h_shared=shared, seed=81)
    check_backward(w, q, k, v, h, seed=81, direct=int(np.prod(dims)) <= 512)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("shared", [False, True])
@pytest.mark.parametrize("dims", [(64,), (16, 32), (4, 8, 16)], ids=str)
def test_backward_circular(dims, shared, dtype):
    w, (q, k, v, h) = W.random_problem(dims, B=2, C=3, dtype=dtype, h_shared=shared, seed=82, circular=True)
    check_backward(w, q, k, v, h, seed=82)


@pytest.mark.parametrize("causal", [True, False])
def test_backward_long_1d(causal):
    """Padded length above one shared-memory line: the kernel gradient comes from causal convolutions of reversed signals."""
    w, (q, k, v, h) = W.random_problem((40000,), B=2, C=2, dtype="bf16", causal=causal, h_shared=True, seed=83)
    check_backward(w, q, k, v, h, seed=83)
    w, (q, k, v, h) = W.random_problem((20000,), B=1, C=2, dtype="f32", causal=causal, seed=84)
    check_backward(w, q, k, v, h, seed=84)


@pytest.mark.parametrize("shared", [False, True])
@pytest.mark.parametrize("dims,causal,dtype", [((33, 20), False, "bf16"), ((40, 50), False, "bf16"), ((40, 48), False, "f32"),
                                               ((6, 36, 40), False, "bf16"), ((5, 33, 20), False, "f32"),
                                               ((16384,), True, "bf16"), ((9001,), True, "bf16")], ids=str)
def test_backward_in_several_passes(dims, causal, dtype, shared, monkeypatch):
    """Groups of batch entries (ragged last group) and groups of slices in the kernel-gradient correlation, on every
    path: general N-D, fused 2-D (two gated results of one forward), plane-fused 3-D, long causal 1-D on both kernel
    families (the shared filter's spectrum kept between two forwards, tensors read in the caller's type)."""
    monkeypatch.setenv("HYENAND_BACKWARD_MAX_BATCH", "2")
    monkeypatch.setenv("HYENAND_BACKWARD_RING_SLICES", "5")
    w, (q, k, v, h) = W.random_problem(dims, B=5, C=4, dtype=dtype, causal=causal, h_shared=shared, seed=85)
    check_backward(w, q, k, v, h, seed=85)


def test_backward_rejects_overlapping_tensors():
    """A gradient that overlaps an input or another gradient is refused before anything is launched."""
    from paper_2607_19378_b200 import hyenand as hn
    w, (q, k, v, h) = W.random_problem((15, 14), B=2, C=3, dtype="f32", seed=86)
    bw = hn.Backward(w.dims, w.B, w.C, dtype=w.torch_dtype)
    try:
        dq_, dk_, dv_, dh_ = (t.cuda() for t in (q, k, v, h))
        ddy = torch.ones_like(dq_)
        stride = w.C * h[0, 0].numel()
        n = dq_.numel()
        big = torch.full((2 * n,), 7.0, device="cuda")
        g0, g1, g2, gh = big[:n].view_as(dq_), torch.full_like(dq_, 7.0), torch.full_like(dq_, 7.0), torch.full_like(dh_, 7.0)
        for outs in [(dq_, g1, g2, gh),                                 # dq is q itself
                     (g0, big[4:4 + n].view_as(dq_), g2, gh)]:          # dk overlaps dq
            with pytest.raises(hn.HyenaNDError) as ei:
                hn.hyenand_backward(bw.handle, dq_, dk_, dv_, dh_, stride, ddy, *outs)
            assert ei.value.code == 1 and hn.hyenand_last_error()
        torch.cuda.synchronize()
        assert bool((big == 7.0).all()) and bool((g1 == 7.0).all()) and bool((gh == 7.0).all()), "a rejected call wrote a gradient"
        assert torch.equal(dq_.cpu(), q)
    finally:
        bw.close()
