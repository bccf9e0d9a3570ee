"""GPU parity at the full benchmark sizes, in the launch configuration bench.py times: the
oracle evaluates the defining sum (O1) at seeded sample positions of a few whole slices; the
whole output must be finite."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_19378_b200 import workloads as W

pytestmark = pytest.mark.gpu

TOL = {"f32": 1e-5, "bf16": 2e-3}
SAMPLES_PER_SLICE = 48


@pytest.mark.parametrize("name", ["tiny2d", "genomics1d", "vision2d", "pde2d", "volume3d"])
def test_named_workload_at_full_size(name):
    from paper_2607_19378_b200 import hyenand as hn
    w = W.WORKLOADS[name]
    dev = torch.device("cuda", 0)
    q, k, v, h = W.make_inputs(w, device=dev)
    plan = hn.Plan(w.dims, w.B, w.C, causal=w.causal, dtype=w.torch_dtype)
    y = torch.full_like(q, float("nan"))
    plan.forward(q, k, v, h, y)
    torch.cuda.synchronize()
    status = hn.hyenand_plan_device_status(plan.handle)
    plan.close()
    assert status == 0, "a kernel gave up a bounded wait"
    assert bool(torch.isfinite(y.float()).all()), "non-finite output"
    S = w.B * w.C
    rng = np.random.default_rng(w.seed)
    slices = sorted({0, S // 2, S - 1} | set(int(s) for s in rng.integers(0, S, size=3)))
    L = int(np.prod(w.dims))
    mode = "causal" if w.causal else "linear"
    got, ref = [], []
    for s in slices:
        b, c = divmod(s, w.C)
        hs = h[c] if w.h_shared else h[b, c]
        qs, ks, vs = (t[b, c].cpu()[None, None] for t in (q, k, v))
        idx = rng.integers(0, L, size=SAMPLES_PER_SLICE)
        ref.append(oracle.conv_direct_at(qs, ks, vs, hs.cpu()[None, None], idx, mode))
        got.append(oracle.to_f64(y[b, c].reshape(-1)[torch.from_numpy(idx).to(dev)]))
    got, ref = np.concatenate(got), np.concatenate(ref)
    err = float(np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-300))
    tol = TOL[w.dtype]
    if w.dtype == "bf16":
        # a few hundred samples: allow the sampling fluctuation of the output rounding itself
        rounding = float(np.linalg.norm(torch.from_numpy(ref).bfloat16().double().numpy() - ref) / np.linalg.norm(ref))
        assert err <= 1.1 * rounding + 1e-6, f"{name}: {err:.3e} vs rounding {rounding:.3e}"
        tol = max(tol, 1.1 * rounding)
    assert err <= tol, f"{name}: sampled rel-L2 {err:.3e}"
