"""CPU-only checks of the boundary: the C library loads, exports every symbol the
header declares, and rejects bad arguments without touching a GPU."""
import ctypes
import os
import re

import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "hyenand.h")


@pytest.fixture(scope="module")
def lib():
    from paper_2607_19378_b200.build import build
    path = build()
    from paper_2607_19378_b200 import hyenand as hn
    assert hn.LIB_PATH == path
    return hn


def declared_symbols():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(hyenand_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(lib):
    names = declared_symbols()
    assert "hyenand_create_plan" in names and "hyenand_forward" in names and "hyenand_destroy_plan" in names
    cdll = ctypes.CDLL(lib.LIB_PATH)
    for n in names:
        assert hasattr(cdll, n), f"{n} declared in hyenand.h but not exported"
    for n in names:
        assert hasattr(lib, n), f"binding lacks {n}"


def test_create_plan_rejects_bad_arguments(lib):
    bad = [
        (0, (4,), 1, 1, 0, 0, lib.HYENAND_ERR_INVALID_ARG),
        (4, (4, 4, 4, 4), 1, 1, 0, 0, lib.HYENAND_ERR_INVALID_ARG),
        (1, (0,), 1, 1, 0, 0, lib.HYENAND_ERR_INVALID_ARG),
        (2, (4, -1), 1, 1, 0, 0, lib.HYENAND_ERR_INVALID_ARG),
        (1, (4,), 0, 1, 0, 0, lib.HYENAND_ERR_INVALID_ARG),
        (1, (4,), 1, 0, 0, 0, lib.HYENAND_ERR_INVALID_ARG),
        (1, (4,), 1, 1, 0, 7, lib.HYENAND_ERR_INVALID_ARG),
        (1, (4,), 1, 1, 2, 0, lib.HYENAND_ERR_INVALID_ARG),
        (2, (4, 4), 1, 1, 1, 0, lib.HYENAND_ERR_UNSUPPORTED),
        (2, (8192, 8), 1, 1, 0, 0, lib.HYENAND_ERR_UNSUPPORTED),
    ]
    for ndim, dims, B, C, causal, dtype, code in bad:
        with pytest.raises(lib.HyenaNDError) as e:
            lib.hyenand_create_plan(ndim, dims, B, C, causal, dtype)
        assert e.value.code == code, (ndim, dims, B, C, causal, dtype, str(e.value))
        assert lib.hyenand_last_error() != ""


def test_null_plan_is_rejected_everywhere(lib):
    L = lib.lib()
    assert L.hyenand_forward(None, 16, 16, 16, 16, 16, None) == lib.HYENAND_ERR_INVALID_ARG
    assert L.hyenand_forward_ex(None, 16, 16, 16, 16, 0, 16, None) == lib.HYENAND_ERR_INVALID_ARG
    assert L.hyenand_forward_host(None, 16, 16, 16, 16, 0, 16, None) == lib.HYENAND_ERR_INVALID_ARG
    assert L.hyenand_plan_workspace_bytes(None) == 0
    assert L.hyenand_plan_launches(None, 0) == 0
    L.hyenand_destroy_plan(None)


def test_cufft_composition_reference_matches_oracle():
    """The library-composition reference point of bench.py computes the same operator as the oracle
    (checked on host tensors; on the GPU machine it is only timed beside the product path)."""
    import dataclasses
    import bench
    import oracle
    from paper_2607_19378_b200 import workloads as W
    cases = [W.WORKLOADS["tiny2d"],
             dataclasses.replace(W.WORKLOADS["genomics1d"], dims=(200,), B=2, C=3),
             dataclasses.replace(W.WORKLOADS["volume3d"], dims=(6, 5, 7), B=1, C=2, dtype="f32")]
    for w in cases:
        q, k, v, h = W.make_inputs(w, device="cpu")
        yref = oracle.conv_fft(oracle.to_f64(q), oracle.to_f64(k), oracle.to_f64(v), oracle.to_f64(h),
                               mode="causal" if w.causal else "linear")
        y = torch.from_numpy(yref).to(q.dtype)
        r = bench.cufft_composition(w, (q, k, v, h, y), reps=1)
        assert r["rel_l2_vs_ours_first_16M"] < (1e-5 if w.dtype == "f32" else 4e-3), (w.name, r)
