"""Parity on seeded random shapes: sizes, dtypes, layouts, epilogues and output types drawn
from a fixed seed, the plan left to choose its own kernel, tile and K split; every result is
compared element by element with the CPU oracle under the acceptance bound."""
import numpy as np
import pytest

import nk_inputs
from nk_testlib import run_and_check

pytestmark = pytest.mark.gpu


def _cases():
    rng = np.random.default_rng(20251113764)
    out = []
    for i in range(36):
        dt = "bf16" if i % 3 else "f32"
        layout = "blocked32" if (dt == "bf16" and i % 6 == 1) else "row"
        step = 32 if layout == "blocked32" else (8 if dt == "bf16" else 4)
        M = int(rng.integers(1, 700))
        N = int(rng.integers(1, 160)) * step
        K = int(rng.integers(1, 260)) * step
        if layout == "blocked32":
            M = max(32, M // 32 * 32)
        epi = "bias_relu" if rng.integers(0, 2) else "none"
        out_dt = "bf16" if (dt == "bf16" and rng.integers(0, 2)) else "f32"
        out.append(nk_inputs.Workload(f"rnd{i}_{dt}_{layout}_{M}x{N}x{K}_{epi}_{out_dt}", M, N, K, dt, out_dt,
                                      layout, epi, dist_a=("normal", 1.0), dist_b=("uniform", 1.0),
                                      seed=9000 + i))
    return out


@pytest.mark.parametrize("w", _cases(), ids=lambda w: w.name)
def test_random_shape(w):
    run_and_check(w)


# ---------------------------------------------------------------- the other operand types and forms, plan on auto
def _extended_cases():
    """Seeded draws over what the first list leaves out: FP16, INT8 (bit-exact), E4M3 / E5M2, B kept as its
    transpose, beta = 1 and batch-reduce with 2 or 3 items; odd sizes, the plan chooses everything."""
    rng = np.random.default_rng(2511137640)
    kinds = ["f16_row", "f16_blocked", "f16_bt", "bf16_bt", "s8_blocked", "s8_bt", "e4m3_blocked", "e5m2_blocked",
             "e4m3_bt", "beta_bf16", "beta_f32", "batch_bf16", "batch_f32"]
    out = []
    for i in range(39):
        kind = kinds[i % len(kinds)]
        M = int(rng.integers(1, 600))
        eight_bit = kind.startswith(("s8", "e4m3", "e5m2"))
        step_n = 32 if (eight_bit or kind == "f16_blocked") else 8
        step_k = 32 if (eight_bit or kind == "f16_blocked") else 16 if kind.endswith("_bt") else 8
        N = int(rng.integers(1, 1200 // step_n)) * step_n
        K = int(rng.integers(1, 2400 // step_k)) * step_k
        if kind == "f16_blocked":
            M = max(32, M // 32 * 32)
        if kind.endswith("_f32"):
            N, K = max(4, N // 4 * 4), max(4, K // 4 * 4)
        epi = bool(rng.integers(0, 2))
        narrow_out = bool(rng.integers(0, 2))
        batch = int(rng.integers(2, 4)) if kind.startswith("batch") else 1
        if batch > 1:
            K = max(step_k, K // 2 // step_k * step_k)
        out.append(pytest.param(kind, M, N, K, epi, narrow_out, batch, 9100 + i, id=f"x{i}_{kind}_{M}x{N}x{K}_b{batch}"))
    return out


def _run_beta_or_batch(dt, M, N, K, batch, beta, epi, narrow_out, seed):
    import torch
    import oracle
    import paper_2511_13764_b200 as nk
    from nk_testlib import to_device, c_to_f64, TOL_REL_SMAX, TOL_BF16_REL
    out_dt = "bf16" if (dt == "bf16" and narrow_out) else "f32"
    pad_a, pad_b = (64, 8) if batch > 1 else (0, 0)
    sa, sb = M * K + pad_a, K * N + pad_b
    A = nk_inputs.fill(seed, nk_inputs.TENSOR_A, (batch - 1) * sa + M * K, "normal", 1.0, dt)
    B = nk_inputs.fill(seed, nk_inputs.TENSOR_B, (batch - 1) * sb + K * N, "uniform", 1.0, dt)
    bias = nk_inputs.fill(seed, nk_inputs.TENSOR_BIAS, N, "normal", 0.5, dt) if epi else None
    C0 = nk_inputs.fill(seed, 5, M * N, "uniform", 1.0, out_dt)
    plan = nk.Plan(M, N, K, nk.BF16 if dt == "bf16" else nk.F32, nk.BF16 if out_dt == "bf16" else nk.F32,
                   epilogue=nk.EPI_BIAS_RELU if epi else nk.EPI_NONE, beta=beta, batch=batch if batch > 1 else 0,
                   stride_a=sa if batch > 1 else 0, stride_b=sb if batch > 1 else 0)
    dC = to_device(C0).clone()
    ws = torch.empty(max(plan.workspace_bytes, 16), dtype=torch.uint8, device="cuda")
    plan.run(to_device(A), to_device(B), dC, bias=to_device(bias) if epi else None,
             workspace=ws if plan.workspace_bytes else None, workspace_bytes=plan.workspace_bytes,
             stream=torch.cuda.current_stream().cuda_stream)
    plan.check()
    got = c_to_f64(dC).reshape(M, N)
    c0 = (C0.astype(np.uint32) << 16).view(np.float32) if out_dt == "bf16" else C0
    Y, S = oracle.brgemm(M, N, K, batch, A, B, bias, C0=c0.astype(np.float64).reshape(M, N) if beta else None,
                         in_dtype=oracle.BF16 if dt == "bf16" else oracle.F32,
                         epilogue=oracle.EPI_BIAS_RELU if epi else oracle.EPI_NONE, beta=float(beta), stride_a=sa, stride_b=sb)
    tol = TOL_REL_SMAX * S.max() + (TOL_BF16_REL * np.abs(Y) if out_dt == "bf16" else 0.0)
    bad = np.abs(got - Y) > tol
    assert not bad.any(), f"{plan.kernel_name}: {bad.sum()} of {bad.size} out of tolerance"


def _run_s8(layout, M, N, K, seed):
    import torch
    import oracle
    import paper_2511_13764_b200 as nk
    A = nk_inputs.fill(seed, nk_inputs.TENSOR_A, M * K, dtype="s8")
    B = nk_inputs.fill(seed, nk_inputs.TENSOR_B, K * N, dtype="s8")
    plan = nk.Plan(M, N, K, in_dtype=nk.S8, out_dtype=nk.S32, layout_a=nk.ROW_MAJOR,
                   layout_b=nk.BLOCKED32 if layout == "blocked" else nk.TRANSPOSED)
    C = torch.full((M * N,), 12345, dtype=torch.int32, device="cuda")
    ws = torch.empty(max(plan.workspace_bytes, 16), dtype=torch.uint8, device="cuda")
    plan.run(torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda(), C, workspace=ws if plan.workspace_bytes else None,
             workspace_bytes=plan.workspace_bytes, stream=torch.cuda.current_stream().cuda_stream)
    plan.check()
    want = oracle.gemm_s8(M, N, K, A, B, layout_b=oracle.BLOCKED32 if layout == "blocked" else oracle.TRANSPOSED)
    got = C.cpu().numpy().astype(np.int64).reshape(M, N)
    assert np.array_equal(got, want), plan.kernel_name


@pytest.mark.parametrize("kind,M,N,K,epi,narrow_out,batch,seed", _extended_cases())
def test_random_shape_other_types_and_forms(kind, M, N, K, epi, narrow_out, batch, seed):
    dt, form = kind.split("_")
    if dt == "s8":
        return _run_s8("blocked" if form == "blocked" else "bt", M, N, K, seed)
    if dt in ("beta", "batch"):
        return _run_beta_or_batch(form, M, N, K, batch, 1 if dt == "beta" else int(seed % 2), epi, narrow_out, seed)
    layout = {"row": "row", "blocked": "blocked32" if dt == "f16" else "b_blocked32", "bt": "b_transposed"}[form]
    out_dt = dt if (dt in ("f16", "bf16") and narrow_out) else "f32"
    w = nk_inputs.Workload(f"x_{kind}", M, N, K, dt, out_dt, layout, "bias_relu" if epi else "none",
                           dist_a=("normal", 1.0), dist_b=("uniform", 1.0), seed=seed)
    run_and_check(w)
