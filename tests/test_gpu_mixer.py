"""GPU parity of the full HyenaND operator (Eq. 2): hyenand_mixer_forward through the C ABI against oracle/mixer.py.

Gates: whole-tensor rel-L2 against the unrounded fp64 oracle (1e-5 fp32 I/O; 2e-3 and 1.1 x output rounding for bf16
I/O), plus an element-wise bound.  The last RMSNorm divides a token's channels by their rms, so an absolute fp32
error d in the gated convolution o shows up as about d / rms_token in y: the bound is
    |y - ref| <= R |ref| + 3 C_el |g_out[c]| rms_b(o) / sqrt(mean_c o_token^2 + eps)
with R, C_el of parity_util (output rounding; fp32 transform error relative to a batch entry's rms level)."""
import numpy as np
import pytest
import torch

import oracle
from oracle import mixer as omix
from paper_2607_19378_b200 import workloads as W
from parity_util import ELEM_C, ELEM_R, TOL, assert_guards, guarded_output

pytestmark = pytest.mark.gpu

EPS = 1e-6


def run_mixer(w, q, k, v, h, g_in, g_out, eps=EPS):
    from paper_2607_19378_b200 import hyenand as hn
    mx = hn.Mixer(w.dims, w.B, w.C, mode=w.mode, dtype=w.torch_dtype, eps=eps)
    try:
        dq, dk, dv, dh = (t.cuda() for t in (q, k, v, h))
        big, y = guarded_output(dq)
        mx.forward(dq, dk, dv, dh, g_in.cuda(), g_out.cuda(), y)
        mx.forward(dq, dk, dv, dh, g_in.cuda(), g_out.cuda(), y)      # the scratch keeps nothing that must be cleared
        torch.cuda.synchronize()
        assert hn.hyenand_plan_device_status(hn.hyenand_mixer_plan(mx.handle)) == 0
        assert hn.hyenand_mixer_guard_damage(mx.handle) == 0
        assert_guards(big, dq.numel(), str(w))
        return y.cpu().clone()
    finally:
        mx.close()


def check_mixer(w, q, k, v, h, seed=0, eps=EPS, direct=False):
    g = torch.Generator().manual_seed(seed)
    g_in = (1.0 + 0.3 * torch.randn(w.C, generator=g)).float()
    g_out = (1.0 + 0.3 * torch.randn(w.C, generator=g)).float()
    y = run_mixer(w, q, k, v, h, g_in, g_out, eps)
    ref, gated = omix.hyena_mixer(q, k, v, h, g_in, g_out, eps=eps, mode=w.mode, direct=direct, parts=True)
    err = oracle.rel_l2(y, ref)
    tol = TOL[w.dtype]
    if w.dtype == "bf16":
        rounding = oracle.rel_l2(torch.from_numpy(ref).bfloat16(), ref)
        assert err <= 1.1 * rounding + 1e-6, f"{w}: rel-L2 {err:.3e} vs rounding {rounding:.3e}"
        if ref.size < 4096:
            tol = max(tol, 1.1 * rounding)
    assert np.isfinite(err) and err <= tol, f"{w}: rel-L2 {err:.3e}"
    yd = oracle.to_f64(y)
    tok = np.sqrt(np.mean(gated * gated, axis=1, keepdims=True) + eps)
    level = np.sqrt(np.mean(gated.reshape(w.B, -1) ** 2, axis=1)).reshape((w.B, 1) + (1,) * len(w.dims))
    gshape = (1, w.C) + (1,) * len(w.dims)
    bound = ELEM_R[w.dtype] * np.abs(ref) + 3 * ELEM_C * np.abs(g_out.double().numpy()).reshape(gshape) * level / tok + 1e-37
    ex = float(np.max(np.abs(yd - ref) / bound))
    assert ex <= 1.0, f"{w}: an element is off by {ex:.2f} x its bound"
    return err


SHAPES = [((5,), False), ((300,), False), ((1000,), True), ((40000,), True), ((15, 14), False), ((40, 50), False),
          ((64, 64), False), ((150, 200), False), ((5, 3, 2), False), ((20, 40, 50), False)]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("shared", [False, True])
@pytest.mark.parametrize("dims,causal", SHAPES, ids=str)
def test_mixer_matches_the_oracle(dims, causal, shared, dtype):
    w, (q, k, v, h) = W.random_problem(dims, B=2, C=5, dtype=dtype, causal=causal, h_shared=shared, seed=61)
    check_mixer(w, q, k, v, h, seed=61, direct=int(np.prod(dims)) <= 2048)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_mixer_circular(dtype):
    w, (q, k, v, h) = W.random_problem((32, 64), B=2, C=4, dtype=dtype, seed=62, circular=True)
    check_mixer(w, q, k, v, h, seed=62)


def test_mixer_single_channel_closed_form_and_zero_tokens():
    """C = 1, eps = 0, delta kernel: y = sign(q k) sign(g_in) g_out; and a token whose q is zero in every channel
    gives a zero inner gate there (the l2 floor keeps it finite)."""
    L = 64
    w, (q, k, v, h) = W.random_problem((L,), B=2, C=1, dtype="f32", seed=63)
    h = torch.zeros_like(h)
    h[..., L - 1] = 1.7
    y = run_mixer(w, q, k, v, h, torch.tensor([-0.3]), torch.tensor([2.5]), eps=0.0)
    want = torch.sign(q * k) * -1.0 * 2.5
    assert float((y - want).abs().max()) < 1e-5
    w2, (q2, k2, v2, h2) = W.random_problem((50,), B=1, C=3, dtype="f32", seed=64)
    q2[:, :, 7] = 0.0
    y2 = run_mixer(w2, q2, k2, v2, h2, torch.ones(3), torch.ones(3))
    assert bool(torch.isfinite(y2).all())
    ref = omix.hyena_mixer(q2, k2, v2, h2, np.ones(3), np.ones(3), eps=EPS)
    assert oracle.rel_l2(y2, ref) <= 1e-5


@pytest.mark.parametrize("dtype,shared", [("f32", False), ("bf16", False), ("bf16", True)])
def test_mixer_runs_in_several_passes_over_the_batch(dtype, shared, monkeypatch):
    """A batch whose fp32 scratch would exceed its bound is worked off in groups of batch entries (forced here to
    two entries per pass): per-sample kernels must come from the right batch entry in every pass, the last pass is
    ragged."""
    monkeypatch.setenv("HYENAND_MIXER_MAX_BATCH", "2")
    w, (q, k, v, h) = W.random_problem((33, 20), B=5, C=4, dtype=dtype, h_shared=shared, seed=65)
    check_mixer(w, q, k, v, h, seed=65)
