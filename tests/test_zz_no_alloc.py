"""The forward entry point that allocates no device memory.

Some callers cannot call cudaMalloc when they need the operator (another thread is capturing a
CUDA graph, the caller sits inside its allocator's critical section, or all device memory was
handed out at start-up).  hyenand_forward_noalloc serves them from a fixed 16 MiB array inside the
library.  Here it is called through the C ABI twice in a row; each result is compared with the
regular plan-based entry point on the same inputs and with the CPU oracle, with the gates the parity
tests use, and the device's free memory must not move across the calls."""
import gc

import numpy as np
import pytest
import torch

import oracle
from paper_2607_19378_b200 import workloads as W
from parity_util import TOL, assert_guards, assert_parity, guarded_output

pytestmark = pytest.mark.gpu

CASES = [
    ((32, 32), 2, 3, "f32", False, False),
    ((40, 50), 2, 2, "bf16", False, True),
    ((1000,), 2, 3, "f32", True, True),
    ((5, 12, 9), 1, 2, "f32", False, False),
    ((65, 20, 20), 1, 2, "f32", False, False),      # core axis padded to 256 points (cp.async core)
    ((300, 20), 2, 2, "bf16", False, False),        # core axis padded to 1024 points
    ((128, 256), 4, 6, "f32", False, False),        # 21 slices fit the array: two passes over the batch
    ((128, 256), 9, 6, "f32", False, True),         # shared filter, 51 slices per pass: the second pass starts at channel 3
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
    ref = oracle.conv_fft(q, k, v, h, "causal" if causal else "linear")
    stride = 0 if shared else C * h[0, 0].numel()
    code = hn.HYENAND_F32 if dtype == "f32" else hn.HYENAND_BF16
    big, y = guarded_output(dq)
    hn.hyenand_forward_noalloc(w.dims, B, C, int(causal), code, dq, dk, dv, dh, stride, y)      # warm-up: loads the kernels
    torch.cuda.synchronize()
    for attempt in range(2):
        y.fill_(float("nan"))
        gc.collect()                                            # garbage of earlier tests must not be freed mid-call
        torch.cuda.synchronize()
        before_torch = torch.cuda.memory_allocated()
        free_before, _ = torch.cuda.mem_get_info()              # the driver's own count: sees any cudaMalloc in the process
        hn.hyenand_forward_noalloc(w.dims, B, C, int(causal), code, dq, dk, dv, dh, stride, y)
        torch.cuda.synchronize()
        free_after, _ = torch.cuda.mem_get_info()
        assert torch.cuda.memory_allocated() == before_torch    # torch's allocator was not touched
        assert free_after == free_before, "device memory was allocated or freed during the call"
        assert_guards(big, dq.numel(), f"noalloc call {attempt}")
        err = oracle.rel_l2(y.cpu(), oracle.to_f64(y_ref.cpu()))
        assert np.isfinite(err) and err <= TOL[dtype], f"call {attempt}: rel-L2 vs hyenand_forward_ex {err:.3e}"
        assert_parity(y.cpu(), ref, q, w, what=f"noalloc call {attempt} vs oracle")


def test_noalloc_rejects_what_does_not_fit():
    from paper_2607_19378_b200 import hyenand as hn
    assert hn.hyenand_noalloc_max_bytes() == 16 << 20
    # the size checks come before anything looks at the buffers: five distinct 16-byte-aligned addresses suffice
    t = [torch.zeros((10 << 20) // 4, device="cuda") for _ in range(5)]
    with pytest.raises(hn.HyenaNDError) as e:                   # one 3-D slice of 64^3 needs far more than 16 MiB
        hn.hyenand_forward_noalloc((64, 64, 64), 1, 1, 0, hn.HYENAND_F32, t[0], t[1], t[2], t[3], 127 ** 3, t[4])
    assert e.value.code == hn.HYENAND_ERR_UNSUPPORTED and "bytes" in str(e.value)
    with pytest.raises(hn.HyenaNDError) as e:                   # beyond the per-axis limit
        hn.hyenand_forward_noalloc((8192,), 1, 1, 1, hn.HYENAND_F32, t[0], t[1], t[2], t[3], 8192, t[4])
    assert e.value.code == hn.HYENAND_ERR_UNSUPPORTED


def test_noalloc_rejects_an_output_that_overlaps_an_input():
    from paper_2607_19378_b200 import hyenand as hn
    w, (q, k, v, h) = W.random_problem((15, 14), B=2, C=3, dtype="f32", seed=42)
    dq, dk, dv, dh = (t.cuda() for t in (q, k, v, h))
    big = torch.full((dq.numel() + 8,), 7.0, device="cuda")
    stride = w.C * h[0, 0].numel()
    with pytest.raises(hn.HyenaNDError) as e:                   # y starts 16 bytes into v
        hn.hyenand_forward_noalloc(w.dims, w.B, w.C, 0, hn.HYENAND_F32, dq, dk, big[:dq.numel()], dh, stride,
                                   big[4:4 + dq.numel()])
    assert e.value.code == hn.HYENAND_ERR_INVALID_ARG and "overlaps" in str(e.value)
    torch.cuda.synchronize()
    assert bool((big == 7.0).all()), "a rejected call wrote to y"
