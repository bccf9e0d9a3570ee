"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle on
identical seeded inputs.  Gates (parity_util.py): whole-tensor relative L2 against
the unrounded fp64 oracle, <= 1e-5 for fp32 I/O and <= 2e-3 for bf16 I/O, plus a bound on
every single element; y sits between guard bands that must stay untouched."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_19378_b200 import workloads as W

pytestmark = pytest.mark.gpu

from parity_util import TOL, check, run_gpu


SHAPES_1D = [(1,), (2,), (3,), (5,), (17,), (64,), (200,), (400,), (1000,), (4096,)]
SHAPES_ND = [(3, 5), (15, 14), (32, 32), (33, 70), (64, 64), (1, 9), (9, 1), (150, 200), (300, 129), (100, 40), (128, 512),
             (5, 3, 2), (7, 1, 4), (16, 16, 16), (20, 9, 12), (1, 1, 6)]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("dims", SHAPES_1D + SHAPES_ND, ids=str)
def test_small_shapes_per_sample_filter(dims, dtype):
    w, (q, k, v, h) = W.random_problem(dims, B=2, C=3, dtype=dtype, seed=11)
    check(w, q, k, v, h, full_direct=int(np.prod(dims)) <= 4096)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("dims", [(5,), (64,), (1000,), (15, 14), (5, 3, 2)], ids=str)
def test_filter_shared_over_batch(dims, dtype):
    w, (q, k, v, h) = W.random_problem(dims, B=3, C=2, dtype=dtype, h_shared=True, seed=12)
    assert h.shape[0] == 2
    check(w, q, k, v, h, full_direct=True)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("L", [1, 2, 7, 64, 1000, 4096])
@pytest.mark.parametrize("shared", [False, True])
def test_causal_1d(L, dtype, shared):
    w, (q, k, v, h) = W.random_problem((L,), B=2, C=3, dtype=dtype, causal=True, h_shared=shared, seed=13)
    check(w, q, k, v, h, full_direct=L <= 1000)


PLANE_SHAPES = [(3, 40, 50), (2, 64, 64), (3, 33, 64), (2, 65, 128), (4, 128, 100), (1, 128, 128), (5, 1, 70)]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("dims", PLANE_SHAPES, ids=str)
def test_plane_fused_3d_path(dims, dtype):
    """3-D grids whose two inner padded axes are 128 or 256 take the plane-fused kernels."""
    w, (q, k, v, h) = W.random_problem(dims, B=1, C=2, dtype=dtype, seed=21)
    from paper_2607_19378_b200 import hyenand as hn
    plan = hn.Plan(w.dims, w.B, w.C, dtype=w.torch_dtype)
    path = hn.hyenand_plan_path(plan.handle)
    plan.close()
    if dims[1] == 1:
        assert path == "nd_generic"
    elif dims[0] > 1:
        assert path == "planes3d"
    check(w, q, k, v, h)


FUSED2D_SHAPES = [(20, 30), (17, 32), (33, 64), (40, 50), (63, 33), (64, 64)]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("shared", [False, True])
@pytest.mark.parametrize("dims", FUSED2D_SHAPES, ids=str)
def test_fused_2d_path(dims, dtype, shared):
    """2-D grids whose padded axes are both 64 or both 128 run as one fused kernel."""
    w, (q, k, v, h) = W.random_problem(dims, B=3, C=2, dtype=dtype, h_shared=shared, seed=23)
    from paper_2607_19378_b200 import hyenand as hn
    plan = hn.Plan(w.dims, w.B, w.C, dtype=w.torch_dtype)
    assert hn.hyenand_plan_path(plan.handle) == "fused2d"
    assert hn.hyenand_plan_launches(plan.handle, shared) == 1
    plan.close()
    check(w, q, k, v, h)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("shared", [False, True])
@pytest.mark.parametrize("dims", [(6, 40, 20), (3, 100, 300), (2, 300, 40), (5, 17, 33)], ids=str)
def test_general_3d_path_with_a_long_middle_axis(dims, dtype, shared):
    """3-D grids whose inner padded axes differ run on the general path; a middle axis padded to 64 .. 1024 points
    takes the warp-engine axis kernel (forward with the filter's wrapped placement, pruned forward, cropped inverse)."""
    from paper_2607_19378_b200 import hyenand as hn
    w, (q, k, v, h) = W.random_problem(dims, B=2, C=2, dtype=dtype, h_shared=shared, seed=31)
    plan = hn.Plan(w.dims, w.B, w.C, dtype=w.torch_dtype)
    path = hn.hyenand_plan_path(plan.handle)
    plan.close()
    assert path == "nd_generic"
    check(w, q, k, v, h)


def _seeded_fused_shapes():
    """Eight seeded shapes inside the domains of the plane-fused 3-D and the fused 2-D kernels (both inner padded axes
    equal: extents in (P/4, P/2]), with seeded batch, channel, dtype and filter-sharing choices."""
    g = np.random.default_rng(20261125)
    cases = []
    for i in range(8):
        P = int(g.choice([128, 256] if i < 5 else [64, 128]))
        ly, lx = (int(g.integers(P // 4 + 1, P // 2 + 1)) for _ in range(2))
        dims = (int(g.integers(1, 9)) + 1, ly, lx) if i < 5 else (ly, lx)
        cases.append((dims, int(g.integers(1, 4)), int(g.integers(1, 4)), ["f32", "bf16"][i % 2], bool(g.integers(0, 2))))
    return cases


@pytest.mark.parametrize("dims,B,C,dtype,shared", _seeded_fused_shapes(), ids=str)
def test_seeded_shapes_on_the_fused_paths(dims, B, C, dtype, shared):
    from paper_2607_19378_b200 import hyenand as hn
    w, (q, k, v, h) = W.random_problem(dims, B=B, C=C, dtype=dtype, h_shared=shared, seed=29)
    plan = hn.Plan(w.dims, w.B, w.C, dtype=w.torch_dtype)
    path = hn.hyenand_plan_path(plan.handle)
    plan.close()
    assert path == ("planes3d" if len(dims) == 3 else "fused2d")
    check(w, q, k, v, h)


TMA_CORE_SHAPES = [(70, 40, 50), (128, 33, 64), (65, 64, 64), (100, 65, 70)]


@pytest.mark.parametrize("dtype,shared", [("f32", False), ("bf16", False), ("f32", True)])
@pytest.mark.parametrize("dims", TMA_CORE_SHAPES, ids=str)
def test_plane_fused_3d_with_256_point_depth_axis(dims, dtype, shared):
    """A depth axis padded to 256 points takes the spectral core whose tiles move as tensor (TMA)
    copies; its bounded waits must not have given up (device status 0)."""
    from paper_2607_19378_b200 import hyenand as hn
    w, (q, k, v, h) = W.random_problem(dims, B=2, C=2, dtype=dtype, h_shared=shared, seed=27)
    plan = hn.Plan(w.dims, w.B, w.C, dtype=w.torch_dtype)
    try:
        assert hn.hyenand_plan_path(plan.handle) == "planes3d"
        dq, dk, dv, dh = (t.cuda() for t in (q, k, v, h))
        y = torch.full_like(dq, float("nan"))
        plan.forward(dq, dk, dv, dh, y)
        plan.forward(dq, dk, dv, dh, y)                     # a second pass over the same buffers
        torch.cuda.synchronize()
        assert hn.hyenand_plan_device_status(plan.handle) == 0
    finally:
        plan.close()
    check(w, q, k, v, h)


def test_plane_fused_3d_shared_filter():
    w, (q, k, v, h) = W.random_problem((3, 40, 50), B=3, C=2, dtype="f32", h_shared=True, seed=22)
    check(w, q, k, v, h)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("causal,shared", [(True, True), (True, False), (False, False)])
@pytest.mark.parametrize("L", [8192, 10000, 9001, 40000])
def test_long_1d_path(L, causal, shared, dtype):
    """Sequences beyond one shared-memory line take the two-pass (Cooley-Tukey) 1-D path."""
    w, (q, k, v, h) = W.random_problem((L,), B=2, C=2, dtype=dtype, causal=causal, h_shared=shared, seed=31)
    from paper_2607_19378_b200 import hyenand as hn
    plan = hn.Plan(w.dims, w.B, w.C, causal=causal, dtype=w.torch_dtype)
    assert hn.hyenand_plan_path(plan.handle) == "ct1d"
    plan.close()
    check(w, q, k, v, h)


LONG_FP32 = [(262144, True), (262144, False), (524288, True), (1048576, False), (2097152, True), (8388608, False)]


@pytest.mark.parametrize("L,causal", LONG_FP32, ids=str)
def test_long_1d_fp32_at_large_padded_sizes(L, causal):
    """fp32 I/O (the 1e-5 gate, where twiddle accuracy shows) on padded lengths 2^19, 2^20, 2^21, 2^22 and 2^24 (the limit the header states): the
    inter-pass twiddles of these lengths are the ones most exposed to rounding.  One slice each; the radix-2 fp64
    oracle takes seconds."""
    w, (q, k, v, h) = W.random_problem((L,), B=1, C=1, dtype="f32", causal=causal, seed=33)
    err = check(w, q, k, v, h)
    assert err <= 2e-6, f"fp32 long 1-D error {err:.3e} is far above the engine's usual 3e-7"


def test_long_1d_bf16_above_2_pow_20():
    w, (q, k, v, h) = W.random_problem((1 << 20,), B=1, C=2, dtype="bf16", causal=True, h_shared=True, seed=34)
    check(w, q, k, v, h)


SWITCH_CASES = [
    ("HYENAND_NO_TMA", (70, 40, 50), "planes3d"),          # cp.async core at a 256-point axis
    ("HYENAND_NO_TMA", (300, 20), "nd_generic"),           # cp.async core at a 1024-point axis
    ("HYENAND_NO_TMA", (40000,), "ct1d"),                  # long 1-D column kernels without tensor copies
    ("HYENAND_GENERIC_CORE", (33, 70), "nd_generic"),      # block-wide core
    ("HYENAND_GENERIC_ROWS", (150, 200), "nd_generic"),    # block-wide row kernels
    ("HYENAND_FORCE_GENERIC", (2, 64, 64), "nd_generic"),  # general N-D passes instead of the plane kernels
    ("HYENAND_FORCE_GENERIC", (40, 50), "nd_generic"),     # ... instead of the fused 2-D kernel
    ("HYENAND_FORCE_GENERIC", (40000,), "ct1d"),           # block-wide long 1-D kernels
]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("switch,dims,path", SWITCH_CASES, ids=str)
def test_kernel_variants_behind_the_switches(switch, dims, path, dtype):
    """Every older kernel variant a development switch selects (read once, at plan creation) still meets the
    gates; they are also what the allocation-free entry point and unusual sizes run."""
    from paper_2607_19378_b200 import hyenand as hn
    import os
    w, (q, k, v, h) = W.random_problem(dims, B=2, C=2, dtype=dtype, seed=35)
    os.environ[switch] = "1"
    try:
        plan = hn.Plan(w.dims, w.B, w.C, dtype=w.torch_dtype)
        assert hn.hyenand_plan_path(plan.handle) == path
        plan.close()
    finally:
        del os.environ[switch]
    check(w, q, k, v, h, env={switch: "1"})


GROUP_CASES = [
    ((70, 40, 50), 3, 3, False, "2", "2"),      # plane-fused 3-D, TMA core: 5 groups on 2 lanes, ragged last group
    ((70, 40, 50), 3, 3, True, "2", "3"),       # shared filter: later groups start at channel offsets 2, 1, 0, 2
    ((128, 256), 4, 6, False, "5", "2"),        # generic 2-D
    ((300, 20), 5, 3, True, "4", "3"),          # generic 2-D, 1024-point TMA core, shared filter, offsets 1, 2, 0
    ((20, 9, 12), 2, 5, False, "3", "4"),       # generic 3-D (block-wide axis kernels)
    ((1000,), 3, 7, True, "4", "2"),            # short 1-D, causal=False
]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("dims,B,C,shared,group,lanes", GROUP_CASES, ids=str)
def test_groups_of_slices_on_several_lanes(dims, B, C, shared, group, lanes, dtype):
    """The batch worked off in groups of slices on several lanes (workspace set + stream each): ragged last group,
    a shared filter whose channel offset is non-zero at a group start, results joined back into the caller's stream."""
    from paper_2607_19378_b200 import hyenand as hn
    w, (q, k, v, h) = W.random_problem(dims, B=B, C=C, dtype=dtype, h_shared=shared, seed=36)
    env = {"HYENAND_GROUP_SLICES": group, "HYENAND_LANES": lanes}
    check(w, q, k, v, h, env=env)
    check(w, q, k, v, h, env=env, stream=torch.cuda.Stream())


@pytest.mark.parametrize("dims,dtype,causal", [((40, 48, 72), "bf16", False), ((200, 300), "f32", False),
                                                ((64, 64), "bf16", False), ((65536,), "bf16", True),
                                                ((1000,), "f32", True)], ids=str)
def test_forward_on_a_non_default_stream(dims, dtype, causal):
    """The forward only enqueues on the stream it is given: run on a side stream while the default stream is
    kept busy, it must give the same result."""
    w, (q, k, v, h) = W.random_problem(dims, B=2, C=2, dtype=dtype, causal=causal, seed=37)
    side = torch.cuda.Stream()
    busy = torch.empty(64 << 20, device="cuda")
    for _ in range(4):
        busy.add_(1.0)                       # default-stream work that a wrongly placed kernel would race with
    check(w, q, k, v, h, stream=side)
    torch.cuda.synchronize()


def test_plan_of_another_device_is_rejected():
    """A plan belongs to the device it was created on; a forward issued with another device current returns an
    error instead of launching on foreign workspace pointers.  Needs two visible devices."""
    if torch.cuda.device_count() < 2:
        pytest.skip("one visible device")
    from paper_2607_19378_b200 import hyenand as hn
    w, (q, k, v, h) = W.random_problem((15, 14), B=1, C=2, dtype="f32", seed=38)
    plan = hn.Plan(w.dims, w.B, w.C, dtype=w.torch_dtype)
    try:
        dq, dk, dv, dh = (t.cuda(0) for t in (q, k, v, h))
        y = torch.zeros_like(dq)
        with torch.cuda.device(1):
            with pytest.raises(hn.HyenaNDError) as e:
                plan.forward(dq, dk, dv, dh, y, stream=0)
            assert e.value.code == hn.HYENAND_ERR_INVALID_ARG
    finally:
        plan.close()


CIRCULAR_SHAPES = [(1,), (2,), (64,), (1024,), (8192,), (4, 8), (32, 32), (64, 128), (256, 64), (1, 16), (16, 1),
                   (2, 4, 8), (16, 16, 16), (8, 1, 32), (4, 64, 64)]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("shared", [False, True])
@pytest.mark.parametrize("dims", CIRCULAR_SHAPES, ids=str)
def test_circular_mode(dims, dtype, shared):
    """Periodic boundaries (Section 3.2.1): the filter lives on the grid itself and the transforms run on
    L_n points with nothing padded, pruned or cropped."""
    from paper_2607_19378_b200 import hyenand as hn
    w, (q, k, v, h) = W.random_problem(dims, B=2, C=3, dtype=dtype, h_shared=shared, seed=51, circular=True)
    assert h.shape[-len(dims):] == tuple(dims)
    plan = hn.Plan(w.dims, w.B, w.C, dtype=w.torch_dtype, circular=True)
    assert hn.hyenand_plan_fft_dims(plan.handle, len(dims)) == tuple(dims)
    plan.close()
    check(w, q, k, v, h, full_direct=int(np.prod(dims)) <= 4096)


def test_circular_mode_wraps_around_and_rejects_other_sizes():
    """A shifted delta filter rolls the gated input around the torus (no zero fill at the edges); grids that are
    not powers of two, or longer than one line, are refused."""
    from paper_2607_19378_b200 import hyenand as hn
    dims = (8, 16)
    w, (q, k, v, h) = W.random_problem(dims, B=1, C=2, dtype="f32", seed=52, circular=True)
    h = torch.zeros_like(h)
    h[..., 3, 14] = 1.0                                   # displacement (+3, -2)
    y, _ = run_gpu(w, q, k, v, h)
    expect = q.double() * torch.roll((k * v).double(), shifts=(3, -2), dims=(-2, -1))
    assert oracle.rel_l2(y, expect.numpy()) < 1e-6
    for bad in [(12,), (8, 6), (16384,)]:
        with pytest.raises(hn.HyenaNDError) as e:
            hn.hyenand_create_plan_mode(len(bad), bad, 1, 1, hn.HYENAND_MODE_CIRCULAR, hn.HYENAND_F32)
        assert e.value.code == hn.HYENAND_ERR_UNSUPPORTED
    with pytest.raises(hn.HyenaNDError) as e:
        hn.hyenand_create_plan_mode(1, (8,), 1, 1, 3, hn.HYENAND_F32)
    assert e.value.code == hn.HYENAND_ERR_INVALID_ARG


def test_tiny2d_workload_full():
    w = W.WORKLOADS["tiny2d"]
    q, k, v, h = W.make_inputs(w)
    err = check(w, q, k, v, h, full_direct=True)
    assert err < 2e-6


def test_delta_filter_and_impulse_on_gpu():
    dims = (6, 10)
    w, (q, k, v, h) = W.random_problem(dims, B=1, C=2, dtype="f32", seed=14)
    h = torch.zeros_like(h)
    h[..., dims[0] - 1, dims[1] - 1] = 1.0
    y, _ = run_gpu(w, q, k, v, h)
    assert oracle.rel_l2(y, (q * k * v).double().numpy()) < 1e-6
    # shifted delta: no wrap-around
    h = torch.zeros_like(h)
    h[..., dims[0] - 1 + 2, dims[1] - 1 - 3] = 1.0
    y, _ = run_gpu(w, q, k, v, h)
    u = (k * v).double()
    exp = torch.zeros_like(u)
    exp[..., 2:, :dims[1] - 3] = u[..., :dims[0] - 2, 3:]
    assert oracle.rel_l2(y, (q.double() * exp).numpy()) < 1e-6


def test_causality_on_gpu():
    L = 300
    w, (q, k, v, h) = W.random_problem((L,), B=1, C=2, dtype="f32", causal=True, seed=15)
    y0, _ = run_gpu(w, q, k, v, h)
    k2, v2 = k.clone(), v.clone()
    k2[..., 200:] = 7.0
    v2[..., 200:] = -3.0
    y1, _ = run_gpu(w, q, k2, v2, h)
    scale = y0.abs().max().item()
    assert (y0[..., :200] - y1[..., :200]).abs().max().item() <= 1e-4 * scale


def test_scaled_named_workloads():
    for name, B, C in [("vision2d", 2, 5), ("pde2d", 1, 2), ("volume3d", 1, 1)]:
        w = W.WORKLOADS[name].scaled(B=B, C=C)
        q, k, v, h = W.make_inputs(w)
        check(w, q, k, v, h)


REPEAT_CASES = [
    ((40, 48, 72), 1, 3, "bf16", False),     # plane-fused 3-D, TMA core
    ((200, 300), 2, 2, "f32", False),        # generic 2-D, TMA core
    ((64, 64), 3, 5, "bf16", False),         # fused 2-D
    ((65536,), 2, 4, "bf16", True),          # long 1-D
    ((1000,), 2, 3, "f32", True),            # short 1-D
]


@pytest.mark.parametrize("dims,B,C,dtype,causal", REPEAT_CASES, ids=lambda c: str(c))
def test_repeated_forwards_are_bit_identical(dims, B, C, dtype, causal):
    """No kernel accumulates with atomics or depends on scheduling order: the same plan run three times on the same
    inputs, with another problem run in between on a second plan, returns the same bits each time, and leaves the
    inputs untouched."""
    from paper_2607_19378_b200 import hyenand as hn
    w, (q, k, v, h) = W.random_problem(dims, B=B, C=C, dtype=dtype, causal=causal, seed=31)
    w2, t2 = W.random_problem((33, 70), B=1, C=2, dtype=dtype, seed=32)
    plan = hn.Plan(w.dims, w.B, w.C, causal=w.causal, dtype=w.torch_dtype)
    other = hn.Plan(w2.dims, w2.B, w2.C, dtype=w2.torch_dtype)
    try:
        dq, dk, dv, dh = (t.cuda() for t in (q, k, v, h))
        d2 = [t.cuda() for t in t2]
        outs = []
        for _ in range(3):
            y = torch.full_like(dq, float("nan"))
            plan.forward(dq, dk, dv, dh, y)
            other.forward(*d2, torch.empty_like(d2[0]))
            torch.cuda.synchronize()
            outs.append(y.cpu())
        assert hn.hyenand_plan_device_status(plan.handle) == 0
        for y in outs[1:]:
            assert torch.equal(y.view(torch.uint8), outs[0].view(torch.uint8))
        for d, t in zip((dq, dk, dv, dh), (q, k, v, h)):
            assert torch.equal(d.cpu().view(torch.uint8), t.view(torch.uint8)), "an input was modified"
    finally:
        plan.close()
        other.close()


def test_bounded_wait_runs_out_and_is_reported():
    """The waits of the TMA kernels are bounded polls: a wait on a barrier that nothing ever completes must
    come back and record its code instead of hanging (no fault, no trap: the kernel simply returns)."""
    from paper_2607_19378_b200 import hyenand as hn
    assert hn.hyenand_selftest_bounded_wait(200) == 9
    # the device is still usable afterwards
    assert float(torch.ones(8, device="cuda").sum().item()) == 8.0


def test_forward_rejects_bad_arguments_and_launches_nothing():
    """Host-side precondition checks of the forward calls: a misaligned pointer, an output that overlaps an input,
    a filter stride that is neither 0 nor C*K, a NULL pointer.  Each returns INVALID_ARG and leaves y untouched."""
    from paper_2607_19378_b200 import hyenand as hn
    w, (q, k, v, h) = W.random_problem((15, 14), B=2, C=3, dtype="f32", seed=21)
    plan = hn.Plan(w.dims, w.B, w.C, dtype=w.torch_dtype)
    try:
        dq, dk, dv, dh = (t.cuda() for t in (q, k, v, h))
        big = torch.full((dq.numel() + 8,), 7.0, device="cuda")
        y = big[:dq.numel()].view_as(dq)
        stride = w.C * h[0, 0].numel()

        def rejected(*args):
            with pytest.raises(hn.HyenaNDError) as ei:
                hn.hyenand_forward_ex(plan.handle, *args)
            assert ei.value.code == 1 and hn.hyenand_last_error()
            torch.cuda.synchronize()
            assert bool((big == 7.0).all()), "a rejected call wrote to y"

        rejected(dq, dk, dv, dh, stride, big[1:1 + dq.numel()])         # y 4 bytes off a 16-byte boundary
        rejected(dq, dk, big[4:4 + dq.numel()], dh, stride, y)          # y overlaps v
        rejected(dq, dk, dv, dh, stride - 1, y)                         # stride neither 0 nor C*K
        L = hn.lib()
        assert L.hyenand_forward_ex(plan.handle, dq.data_ptr(), None, dv.data_ptr(), dh.data_ptr(), stride,
                                    y.data_ptr(), None) == 1
        # the same plan still runs a valid call afterwards
        hn.hyenand_forward_ex(plan.handle, dq, dk, dv, dh, stride, y)
        torch.cuda.synchronize()
        assert oracle.rel_l2(y.cpu(), oracle.conv_fft(q, k, v, h, "linear")) <= TOL["f32"]
    finally:
        plan.close()


HOST_CASES = [
    ((512, 512), 2, 8, "f32", False, False),        # generic 2-D, eight groups of two slices
    ((131072,), 4, 64, "bf16", True, True),         # long 1-D, filter shared over the batch
    ((72, 64, 64), 1, 16, "bf16", False, False),    # plane-fused 3-D with the TMA core
    ((64, 64), 16, 128, "bf16", False, False),      # fused 2-D
    ((20, 30), 2, 3, "f32", False, True),           # small: a single group
]


@pytest.mark.parametrize("dims,B,C,dtype,causal,shared", HOST_CASES, ids=str)
def test_host_forward_pipeline_matches_device_forward(dims, B, C, dtype, causal, shared):
    """hyenand_forward_host (host buffers, copies pipelined over groups of slices inside the call) returns
    exactly what hyenand_forward computes on device-resident copies of the same tensors."""
    from paper_2607_19378_b200 import hyenand as hn
    w = W.Workload("host", dims, B, C, dtype, seed=3, causal=causal, h_shared=shared)
    q, k, v, h = W.make_inputs(w, device="cpu")
    plan = hn.Plan(w.dims, w.B, w.C, causal=causal, dtype=w.torch_dtype)
    try:
        dq, dk, dv, dh = (t.cuda() for t in (q, k, v, h))
        y_dev = torch.full_like(dq, float("nan"))
        plan.forward(dq, dk, dv, dh, y_dev)
        torch.cuda.synchronize()
        host = [t.contiguous().pin_memory() for t in (q, k, v, h)]
        y_host = torch.full_like(q, float("nan")).pin_memory()
        plan.forward_host(*host, y_host)
        plan.forward_host(*host, y_host)                    # and again over the same staging buffers
        assert hn.hyenand_plan_device_status(plan.handle) == 0
    finally:
        plan.close()
    assert torch.equal(y_host, y_dev.cpu())


def test_reporting_helpers_and_nvtx_switch(monkeypatch):
    """hyenand_plan_groups reports how a forward schedules the batch; the NVTX switch (a range per kernel launch,
    read at plan creation) does not change results."""
    from paper_2607_19378_b200 import hyenand as hn
    w, (q, k, v, h) = W.random_problem((70, 40, 50), B=3, C=3, dtype="bf16", seed=91)
    monkeypatch.setenv("HYENAND_GROUP_SLICES", "2")
    monkeypatch.setenv("HYENAND_LANES", "3")
    plan = hn.Plan(w.dims, w.B, w.C, dtype=w.torch_dtype)
    assert hn.hyenand_plan_groups(plan.handle) == (2, 3)
    assert hn.hyenand_plan_launches(plan.handle, False) == 5 * 4          # five groups of four kernels
    y0 = plan.forward(q.cuda(), k.cuda(), v.cuda(), h.cuda()).cpu()
    plan.close()
    monkeypatch.setenv("HYENAND_NVTX", "1")
    plan = hn.Plan(w.dims, w.B, w.C, dtype=w.torch_dtype)
    y1 = plan.forward(q.cuda(), k.cuda(), v.cuda(), h.cuda()).cpu()
    plan.close()
    assert torch.equal(y0.view(torch.uint8), y1.view(torch.uint8))
    fused = hn.Plan((32, 32), 1, 2)
    assert hn.hyenand_plan_groups(fused.handle) == (2, 1)
    fused.close()


def test_long_1d_tensor_maps_follow_the_callers_buffers():
    """The long 1-D path encodes tensor maps for the caller's q, k, v, h, y and caches them per thread: calls that
    alternate between two sets of buffers (and a third call with the first set's pointers holding new data) must each
    see their own tensors."""
    from paper_2607_19378_b200 import hyenand as hn
    wa, ta = W.random_problem((65536,), B=1, C=2, dtype="bf16", causal=True, seed=92)
    wb, tb = W.random_problem((65536,), B=1, C=2, dtype="bf16", causal=True, seed=93)
    plan = hn.Plan(wa.dims, wa.B, wa.C, causal=True, dtype=wa.torch_dtype)
    da, db = [t.cuda() for t in ta], [t.cuda() for t in tb]
    ya, yb = torch.empty_like(da[0]), torch.empty_like(db[0])
    for _ in range(2):
        plan.forward(*da, ya)
        plan.forward(*db, yb)
    torch.cuda.synchronize()
    ra, rb = oracle.conv_fft(*ta, "causal"), oracle.conv_fft(*tb, "causal")
    assert oracle.rel_l2(ya.cpu(), ra) <= TOL["bf16"] and oracle.rel_l2(yb.cpu(), rb) <= TOL["bf16"]
    for d, t in zip(da, tb):
        d.copy_(t)                                        # same pointers, other data
    plan.forward(*da, ya)
    torch.cuda.synchronize()
    assert hn.hyenand_plan_device_status(plan.handle) == 0
    plan.close()
    assert oracle.rel_l2(ya.cpu(), rb) <= TOL["bf16"]
