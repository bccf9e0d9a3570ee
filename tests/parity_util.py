"""Helpers of the GPU parity tests: run the CUDA library through its C ABI inside guard bands and compare
with the fp64 oracle, tensor-wide (relative L2, the gate of the task) and element by element.

Gates
  whole tensor   rel-L2 against the UNROUNDED fp64 oracle: <= 1e-5 (fp32 I/O), <= 2e-3 (bf16 I/O); with bf16
                 additionally <= 1.1 x the error of rounding the exact result to bf16 (the one unavoidable error).
  per element    |y - ref| <= R |ref| + C |q| rms(w)   with w = the ungated convolution of the element's slice.
                 The first term is the output rounding (bf16: half an ulp is 2^-9 |ref|, allowed 2^-8; fp32:
                 2^-24, allowed 2^-22).  The second is the fp32 transform arithmetic, whose error is spread
                 evenly over a slice at a level relative to the slice's rms: the measured whole-tensor rel-L2 of
                 the fp32 path is 2e-7 to 3e-7, so one element in 2^27 reaches about 6 sigma = 2e-6 rms; C = 6e-6
                 leaves a factor 3 on top.  No single wrong element (a tile edge, a tail row) fits under it.
"""
import numpy as np
import torch

import oracle

TOL = {"f32": 1e-5, "bf16": 2e-3}
ELEM_R = {"f32": 2.0 ** -22, "bf16": 2.0 ** -8}
ELEM_C = 6e-6
GUARD = 256                     # elements of the guard band on either side of y
SENTINEL = 7.0


def guarded_output(like):
    """y inside a larger tensor: [GUARD sentinels][y, NaN-filled][GUARD sentinels]."""
    n = like.numel()
    big = torch.full((n + 2 * GUARD,), SENTINEL, dtype=like.dtype, device=like.device)
    y = big[GUARD:GUARD + n].view(like.shape)
    y.fill_(float("nan"))
    return big, y


def assert_guards(big, n, what=""):
    lo, hi = big[:GUARD], big[GUARD + n:]
    assert bool((lo == SENTINEL).all()) and bool((hi == SENTINEL).all()), f"{what}: a kernel wrote outside y"


def run_gpu(w, q, k, v, h, stream=None, env=None):
    """One forward of workload w on cuda:0; returns (y on the host, kernel path).  Checks the guard bands around
    y, the guard bands around the plan's workspace and the device status word."""
    import os
    from paper_2607_19378_b200 import hyenand as hn
    old = {}
    for key, val in (env or {}).items():
        old[key] = os.environ.get(key)
        os.environ[key] = val
    try:
        plan = hn.Plan(w.dims, w.B, w.C, causal=w.causal, dtype=w.torch_dtype, circular=w.circular)
    finally:
        for key, val in old.items():
            if val is None:
                os.environ.pop(key, None)
            else:
                os.environ[key] = val
    try:
        dq, dk, dv, dh = (t.cuda() for t in (q, k, v, h))
        big, y = guarded_output(dq)
        if stream is not None:
            stream.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(stream):
                plan.forward(dq, dk, dv, dh, y, stream=stream)
            stream.synchronize()
        else:
            plan.forward(dq, dk, dv, dh, y)
        torch.cuda.synchronize()
        assert hn.hyenand_plan_device_status(plan.handle) == 0, "a kernel gave up a bounded wait"
        assert hn.hyenand_plan_guard_damage(plan.handle) == 0, "a kernel wrote outside the plan's workspace"
        assert_guards(big, dq.numel(), str(w))
        return y.cpu().clone(), hn.hyenand_plan_path(plan.handle)
    finally:
        plan.close()


def elementwise_excess(y, ref, q, dtype, slices):
    """max over elements of |y - ref| / bound (<= 1 passes).  y, q: tensors; ref: fp64 array of the same shape;
    `slices` = number of leading (b,c) slices the arrays hold."""
    yd = oracle.to_f64(y).reshape(slices, -1)
    rd = np.asarray(ref, dtype=np.float64).reshape(slices, -1)
    qd = oracle.to_f64(q).reshape(slices, -1)
    wconv = np.divide(rd, qd, out=np.zeros_like(rd), where=qd != 0)
    rms = np.sqrt(np.mean(wconv * wconv, axis=1, keepdims=True))
    bound = ELEM_R[dtype] * np.abs(rd) + ELEM_C * np.abs(qd) * rms + 1e-37
    return float(np.max(np.abs(yd - rd) / bound))


def assert_parity(y, ref, q, w, what=""):
    """The whole-tensor and the element-wise gates for output y of workload w against the fp64 reference."""
    err = oracle.rel_l2(y, ref)
    tol = TOL[w.dtype]
    if w.dtype == "bf16":
        rounding = oracle.rel_l2(torch.from_numpy(np.asarray(ref)).bfloat16(), ref)
        assert err <= 1.1 * rounding + 1e-6, f"{w} {what}: rel-L2 {err:.3e} vs rounding {rounding:.3e}"
        if np.asarray(ref).size < 4096:
            # on a few dozen elements the rounding error itself fluctuates above 2e-3
            tol = max(tol, 1.1 * rounding)
    assert np.isfinite(err) and err <= tol, f"{w} {what}: rel-L2 {err:.3e}"
    S = w.B * w.C
    yd = oracle.to_f64(y).reshape(S, -1)
    rd = np.asarray(ref).reshape(S, -1)
    per = np.linalg.norm(yd - rd, axis=1) / np.maximum(np.linalg.norm(rd, axis=1), 1e-300)
    assert per.max() <= 4 * tol, f"{w} {what}: worst slice rel-L2 {per.max():.3e}"
    ex = elementwise_excess(y, ref, q, w.dtype, S)
    assert ex <= 1.0, f"{w} {what}: an element is off by {ex:.2f} x its bound"
    return err


def check(w, q, k, v, h, full_direct=False, stream=None, env=None):
    y, path = run_gpu(w, q, k, v, h, stream=stream, env=env)
    ref = (oracle.conv_direct if full_direct else oracle.conv_fft)(q, k, v, h, w.mode)
    return assert_parity(y, ref, q, w, what=f"path={path}")
