"""The forward entry point that allocates no device memory.

Some callers cannot call cudaMalloc when they need the operator (another thread is capturing a
CUDA graph, the caller sits inside its allocator's critical section, or all device memory was
handed out at start-up).  hyenand_forward_noalloc serves them from a fixed 16 MiB array inside the
library.  Here it is called through the C ABI twice in a row and compared with the regular
plan-based entry point on the same inputs, with the tolerances the parity tests use."""
import gc

import numpy as np
import pytest
import torch

import oracle
from paper_2607_19378_b200 import workloads as W

pytestmark = pytest.mark.gpu

TOL = {"f32": 1e-5, "bf16": 2e-3}
CASES = [
    ((32, 32), 2, 3, "f32", False, False),
    ((40, 50), 2, 2, "bf16", False, True),
    ((1000,), 2, 3, "f32", True, True),
    ((5, 12, 9), 1, 2, "f32", False, False),
]


@pytest.mark.parametrize("dims,B,C,dtype,causal,shared", CASES, ids=str)
def test_noalloc_matches_plan_based_forward_twice(dims, B, C, dtype, causal, shared):
    from paper_2607_19378_b200 import hyenand as hn
    w, (q, k, v, h) = W.random_problem(dims, B=B, C=C, dtype=dtype, causal=causal, h_shared=shared, seed=41)
    dq, dk, dv, dh = (t.cuda() for t in (q, k, v, h))
    plan = hn.Plan(w.dims, w.B, w.C, causal=causal, dtype=w.torch_dtype)
    y_ref = plan.forward(dq, dk, dv, dh)
    torch.cuda.synchronize()
    plan.close()
    stride = 0 if shared else C * h[0, 0].numel()
    code = hn.HYENAND_F32 if dtype == "f32" else hn.HYENAND_BF16
    before = torch.cuda.memory_allocated()
    for attempt in range(2):
        y = torch.full_like(dq, float("nan"))
        gc.collect()                                            # garbage of earlier tests must not be freed mid-call
        before = torch.cuda.memory_allocated()
        hn.hyenand_forward_noalloc(w.dims, B, C, int(causal), code, dq, dk, dv, dh, stride, y)
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() == before          # torch's allocator was not touched either
        err = oracle.rel_l2(y.cpu(), oracle.to_f64(y_ref.cpu()))
        assert np.isfinite(err) and err <= TOL[dtype], f"call {attempt}: rel-L2 vs hyenand_forward_ex {err:.3e}"


def test_noalloc_rejects_what_does_not_fit():
    from paper_2607_19378_b200 import hyenand as hn
    assert hn.hyenand_noalloc_max_bytes() == 16 << 20
    t = torch.zeros(64, device="cuda")
    with pytest.raises(hn.HyenaNDError) as e:                   # one 3-D slice of 64^3 needs far more than 16 MiB
        hn.hyenand_forward_noalloc((64, 64, 64), 1, 1, 0, hn.HYENAND_F32, t, t, t, t, 127 ** 3, t)
    assert e.value.code == hn.HYENAND_ERR_UNSUPPORTED and "bytes" in str(e.value)
    with pytest.raises(hn.HyenaNDError) as e:                   # beyond the per-axis limit
        hn.hyenand_forward_noalloc((8192,), 1, 1, 1, hn.HYENAND_F32, t, t, t, t, 8192, t)
    assert e.value.code == hn.HYENAND_ERR_UNSUPPORTED
