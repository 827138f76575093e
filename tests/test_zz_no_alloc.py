"""nk_gemm_run_static: the GEMM for callers that cannot allocate device memory.

A caller inside an allocation-free region (a serving loop that must not stall
on the allocator, a plug-in that is handed buffers and owns no allocator) still
needs split-K plans to work.  The entry point takes the split-K scratch from a
16 MiB array built into the library.  This test runs it through the C ABI twice
in a row, on different inputs, and compares each result with what nk_gemm_run
produces for the same plan with caller-provided scratch (the two share the
kernels and the summation order, so the results must agree bit for bit, which
is inside the tolerance the other tests use) and with the CPU oracle under the
acceptance bound of the parity tests.  It is collected last so that a failure
here cannot hide one elsewhere.
"""
import numpy as np
import pytest
import torch

import nk_inputs
import paper_2511_13764_b200 as nk
from nk_testlib import to_device, c_to_f64, check_against_oracle, TOL_REL_SMAX

pytestmark = pytest.mark.gpu


def _run_both(plan, w, seed):
    import dataclasses
    A, B, bias = dataclasses.replace(w, seed=seed).make()
    dA, dB = to_device(A), to_device(B)
    db = to_device(bias) if bias is not None else None
    out_dt = torch.float32 if w.out_dtype == "f32" else torch.bfloat16
    sp = torch.cuda.current_stream().cuda_stream
    ws = torch.empty(plan.workspace_bytes, dtype=torch.uint8, device="cuda")
    ref = torch.full((w.M * w.N,), float("nan"), dtype=out_dt, device="cuda")
    plan.run(dA, dB, ref, bias=db, workspace=ws, stream=sp)
    got = torch.full((w.M * w.N,), float("nan"), dtype=out_dt, device="cuda")
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    allocs_before = torch.cuda.memory_stats().get("allocation.all.allocated", 0)
    plan.run_static(dA, dB, got, bias=db, stream=sp)
    plan.check()
    # nothing was allocated on the device: neither through torch's allocator nor behind its back
    assert torch.cuda.memory_stats().get("allocation.all.allocated", 0) == allocs_before
    assert torch.cuda.mem_get_info()[0] >= free_before
    # the static-scratch result against the oracle, element by element, under the acceptance bound
    check_against_oracle(w, c_to_f64(got).reshape(w.M, w.N), A, B, bias)
    return c_to_f64(got), c_to_f64(ref)


@pytest.mark.parametrize("kind", ["bf16_splitk", "f32_splitk"])
def test_static_scratch_matches_caller_scratch_twice(kind):
    if kind == "bf16_splitk":
        w = nk_inputs.Workload("noalloc", 200, 328, 1096, "bf16", "bf16", epilogue="bias_relu", seed=21)
        plan = nk.plan_for(w, flags=nk.flag_splitk(5))
    else:
        w = nk_inputs.Workload("noalloc", 100, 200, 1000, "f32", "f32", seed=22)
        plan = nk.plan_for(w, flags=nk.flag_splitk(4))
    assert 0 < plan.workspace_bytes <= nk.STATIC_SCRATCH_BYTES
    for call, seed in enumerate((31, 32)):          # two calls in a row, different inputs
        got, ref = _run_both(plan, w, seed)
        assert not np.isnan(got).any()
        scale = max(np.abs(ref).max(), 1.0)
        assert np.max(np.abs(got - ref)) <= TOL_REL_SMAX * scale, f"call {call}"
        assert np.array_equal(got, ref), f"call {call}"


def test_static_scratch_rejects_oversized_plans():
    w = nk_inputs.Workload("big", 2048, 2048, 1024, "f32", "f32", seed=23)
    plan = nk.plan_for(w, flags=nk.flag_splitk(2))      # 2 x 16 MiB of partials
    assert plan.workspace_bytes > nk.STATIC_SCRATCH_BYTES
    x = torch.zeros(2048 * 2048, dtype=torch.float32, device="cuda")
    with pytest.raises(nk.NkError) as e:
        plan.run_static(x, x, x)
    assert e.value.status == 4 and "scratch" in str(e.value)


def test_static_entry_without_scratch_need():
    w = nk_inputs.Workload("plain", 128, 256, 256, "bf16", "f32", seed=24)
    plan = nk.plan_for(w)
    assert plan.workspace_bytes == 0
    A, B, _ = w.make()
    dA, dB = to_device(A), to_device(B)
    c1 = torch.empty(w.M * w.N, dtype=torch.float32, device="cuda")
    c2 = torch.empty_like(c1)
    sp = torch.cuda.current_stream().cuda_stream
    plan.run(dA, dB, c1, stream=sp)
    plan.run_static(dA, dB, c2, stream=sp)
    plan.check()
    assert torch.equal(c1, c2)
