"""Batch-reduce GEMM through the C ABI: C = beta*C + sum_b A_b.B_b (Algorithm 1's output
line), with non-contiguous batch items and the fused epilogue, against the oracle's
definition.  Integer-valued data makes the FP32 results exact."""
import numpy as np
import pytest
import torch

import nk_inputs
import oracle
import paper_2511_13764_b200 as nk
from nk_testlib import to_device, c_to_f64, TOL_REL_SMAX, TOL_BF16_REL

pytestmark = pytest.mark.gpu


def _run(M, N, K, batch, dt, out_dt, epi, beta, pad_a=0, pad_b=0, flags=0, integer=True, seed=1):
    sa, sb = M * K + pad_a, K * N + pad_b
    na, nb = (batch - 1) * sa + M * K, (batch - 1) * sb + K * N
    dist = "int" if integer else "uniform"
    A = nk_inputs.fill(seed, nk_inputs.TENSOR_A, na, dist, dtype=dt)
    B = nk_inputs.fill(seed, nk_inputs.TENSOR_B, nb, dist, dtype=dt)
    bias = nk_inputs.fill(seed, nk_inputs.TENSOR_BIAS, N, dist, dtype=dt) if epi else None
    C0 = nk_inputs.fill(seed, 5, M * N, dist, dtype=out_dt)
    plan = nk.Plan(M, N, K, nk.BF16 if dt == "bf16" else nk.F32, nk.BF16 if out_dt == "bf16" else nk.F32,
                   epilogue=nk.EPI_BIAS_RELU if epi else nk.EPI_NONE, flags=flags, beta=beta, batch=batch,
                   stride_a=sa if pad_a else 0, stride_b=sb if pad_b else 0)
    dA, dB = to_device(A), to_device(B)
    dbias = to_device(bias) if epi else None
    dC = to_device(C0).clone()
    ws = torch.empty(max(plan.workspace_bytes, 16), dtype=torch.uint8, device="cuda")
    plan.run(dA, dB, dC, bias=dbias, workspace=ws if plan.workspace_bytes else None,
             workspace_bytes=plan.workspace_bytes, stream=torch.cuda.current_stream().cuda_stream)
    plan.check()
    got = c_to_f64(dC).reshape(M, N)
    c0 = (C0.astype(np.uint32) << 16).view(np.float32) if out_dt == "bf16" else C0
    Y, S = oracle.brgemm(M, N, K, batch, A, B, bias, C0=c0.astype(np.float64).reshape(M, N) if beta else None,
                         in_dtype=oracle.BF16 if dt == "bf16" else oracle.F32,
                         epilogue=oracle.EPI_BIAS_RELU if epi else oracle.EPI_NONE, beta=float(beta),
                         stride_a=sa, stride_b=sb)
    if integer and out_dt == "f32":
        assert np.array_equal(got, Y), plan.kernel_name
    else:
        tol = TOL_REL_SMAX * S.max() + (TOL_BF16_REL * np.abs(Y) if out_dt == "bf16" else 0.0)
        assert np.all(np.abs(got - Y) <= tol), plan.kernel_name
    return plan


# the paper's example kernels: Listing 1 (4 x (32x32).(32x192)), appendix FP32 (2 x (4x32).(32x96)),
# appendix BF16 (2 x (64x64).(64x64))
@pytest.mark.parametrize("M,N,K,batch,dt", [(32, 192, 32, 4, "bf16"), (4, 96, 32, 2, "f32"), (64, 64, 64, 2, "bf16")])
@pytest.mark.parametrize("beta", [0, 1])
def test_paper_example_brgemm_shapes(M, N, K, batch, dt, beta):
    plan = _run(M, N, K, batch, dt, "f32", False, beta)
    assert f"_br{batch}" in plan.kernel_name


@pytest.mark.parametrize("mode", ["single", "pair"])
@pytest.mark.parametrize("beta", [0, 1])
@pytest.mark.parametrize("out_dt,epi", [("f32", False), ("f32", True), ("bf16", True)])
def test_brgemm_bf16(mode, beta, out_dt, epi):
    f = nk.FLAG_SINGLE_CTA if mode == "single" else nk.FLAG_CTA_PAIR
    _run(200, 328, 136, 5, "bf16", out_dt, epi, beta, pad_a=64, pad_b=8, flags=f)           # K tail inside every item
    _run(300, 256, 64, 3, "bf16", out_dt, epi, beta, flags=f | nk.flag_splitk(2), integer=False, seed=3)


@pytest.mark.parametrize("beta", [0, 1])
@pytest.mark.parametrize("tile", [1, 2, 3])
def test_brgemm_f32(beta, tile):
    _run(130, 260, 40, 4, "f32", "f32", True, beta, pad_a=12, pad_b=4, flags=nk.FLAG_KERNEL_SIMT | nk.flag_tile_n(tile))
    _run(100, 200, 100, 3, "f32", "f32", False, beta, flags=nk.flag_tile_n(tile) | nk.flag_splitk(3), integer=False, seed=4)


def test_brgemm_naive_cross_check():
    _run(40, 48, 24, 3, "bf16", "f32", True, 1, pad_a=8, flags=nk.FLAG_KERNEL_NAIVE)
    _run(40, 48, 24, 3, "f32", "f32", False, 1, pad_b=4, flags=nk.FLAG_KERNEL_NAIVE)


def test_beta_one_plain_gemm_auto():
    _run(512, 512, 1024, 1, "bf16", "f32", False, 1, integer=False, seed=5)
    _run(16, 1024, 512, 1, "f32", "f32", False, 1)          # M <= 32 with beta goes to the tiled kernel


# ---------------------------------------------------------------- batched matmul: C_g = A_g . B_g
def _run_bmm(M, N, K, gemms, dt, out_dt, epi, beta, pad_a=0, pad_b=0, pad_c=0, flags=0, integer=True, seed=2):
    sa, sb, sc = M * K + pad_a, K * N + pad_b, M * N + pad_c
    dist = "int" if integer else "uniform"
    A = nk_inputs.fill(seed, nk_inputs.TENSOR_A, (gemms - 1) * sa + M * K, dist, dtype=dt)
    B = nk_inputs.fill(seed, nk_inputs.TENSOR_B, (gemms - 1) * sb + K * N, dist, dtype=dt)
    bias = nk_inputs.fill(seed, nk_inputs.TENSOR_BIAS, N, dist, dtype=dt) if epi else None
    C0 = nk_inputs.fill(seed, 5, (gemms - 1) * sc + M * N, dist, dtype=out_dt)
    plan = nk.Plan(M, N, K, nk.BF16 if dt == "bf16" else nk.F32, nk.BF16 if out_dt == "bf16" else nk.F32,
                   epilogue=nk.EPI_BIAS_RELU if epi else nk.EPI_NONE, flags=flags, beta=beta, batch=gemms,
                   stride_a=sa if pad_a else 0, stride_b=sb if pad_b else 0, stride_c=sc if pad_c else 0,
                   batch_independent=1)
    assert f"_bmm{gemms}" in plan.kernel_name
    dA, dB = to_device(A), to_device(B)
    dbias = to_device(bias) if epi else None
    dC = to_device(C0).clone()
    ws = torch.empty(max(plan.workspace_bytes, 16), dtype=torch.uint8, device="cuda")
    plan.run(dA, dB, dC, bias=dbias, workspace=ws if plan.workspace_bytes else None,
             workspace_bytes=plan.workspace_bytes, stream=torch.cuda.current_stream().cuda_stream)
    plan.check()
    got = c_to_f64(dC)
    c0 = ((C0.astype(np.uint32) << 16).view(np.float32) if out_dt == "bf16" else C0).astype(np.float64)
    for g in range(gemms):
        Y, S = oracle.brgemm(M, N, K, 1, A[g * sa:g * sa + M * K], B[g * sb:g * sb + K * N], bias,
                             C0=c0[g * sc:g * sc + M * N].reshape(M, N) if beta else None,
                             in_dtype=oracle.BF16 if dt == "bf16" else oracle.F32,
                             epilogue=oracle.EPI_BIAS_RELU if epi else oracle.EPI_NONE, beta=float(beta))
        gg = got[g * sc:g * sc + M * N].reshape(M, N)
        if integer and out_dt == "f32":
            assert np.array_equal(gg, Y), (plan.kernel_name, g)
        else:
            tol = TOL_REL_SMAX * S.max() + (TOL_BF16_REL * np.abs(Y) if out_dt == "bf16" else 0.0)
            assert np.all(np.abs(gg - Y) <= tol), (plan.kernel_name, g)
    if pad_c:   # the gaps between the C's are untouched
        for g in range(gemms - 1):
            assert np.array_equal(got[g * sc + M * N:(g + 1) * sc], c0[g * sc + M * N:(g + 1) * sc])
    return plan


@pytest.mark.parametrize("mode", ["single", "pair"])
@pytest.mark.parametrize("beta", [0, 1])
def test_batched_matmul_bf16(mode, beta):
    f = nk.FLAG_SINGLE_CTA if mode == "single" else nk.FLAG_CTA_PAIR
    _run_bmm(200, 136, 72, 5, "bf16", "f32", False, beta, pad_a=8, pad_b=16, pad_c=12, flags=f)
    _run_bmm(130, 256, 192, 3, "bf16", "bf16", True, beta, flags=f | nk.flag_splitk(3), integer=False)


@pytest.mark.parametrize("beta", [0, 1])
@pytest.mark.parametrize("tile", [1, 2, 3])
def test_batched_matmul_f32(beta, tile):
    _run_bmm(70, 132, 52, 4, "f32", "f32", True, beta, pad_a=4, pad_c=8, flags=nk.FLAG_KERNEL_SIMT | nk.flag_tile_n(tile))
    _run_bmm(64, 64, 256, 6, "f32", "f32", False, beta, flags=nk.flag_tile_n(tile) | nk.flag_splitk(2), integer=False)


def test_batched_matmul_auto_and_naive():
    _run_bmm(256, 256, 256, 16, "bf16", "f32", False, 0, integer=False)
    _run_bmm(24, 40, 16, 3, "f32", "f32", True, 1, pad_c=4, flags=nk.FLAG_KERNEL_NAIVE)
    _run_bmm(16, 64, 64, 4, "f32", "f32", False, 0)      # small M, batched: tiled kernel, not the streaming one


# ---------------------------------------------------------------- batch items in the blocked / VNNI-packed layout
def _run_layout(M, N, K, batch, out_dt, epi, beta, layout, pad_a=0, pad_b=0, flags=0, integer=True, seed=1,
                independent=False):
    """Batch items stored blocked (A[M/32][K/32][32][32], B VNNI-packed [N/32][K/32][16][32][2]) or with B kept
    as its transpose; entries are i.i.d., so a buffer of the right length filled by index is a valid operand
    in any layout.  Compared with the oracle's layout-aware batch-reduce."""
    sa, sb = M * K + pad_a, K * N + pad_b
    dist = "int" if integer else "uniform"
    A = nk_inputs.fill(seed, nk_inputs.TENSOR_A, (batch - 1) * sa + M * K, dist, dtype="bf16")
    B = nk_inputs.fill(seed, nk_inputs.TENSOR_B, (batch - 1) * sb + K * N, dist, dtype="bf16")
    bias = nk_inputs.fill(seed, nk_inputs.TENSOR_BIAS, N, dist, dtype="bf16") if epi else None
    C0 = nk_inputs.fill(seed, 5, M * N, dist, dtype=out_dt)
    lay_a = nk.BLOCKED32 if layout == "blocked" else nk.ROW_MAJOR
    lay_b = nk.BLOCKED32 if layout == "blocked" else nk.TRANSPOSED
    plan = nk.Plan(M, N, K, nk.BF16, nk.BF16 if out_dt == "bf16" else nk.F32, layout_a=lay_a, layout_b=lay_b,
                   epilogue=nk.EPI_BIAS_RELU if epi else nk.EPI_NONE, flags=flags, beta=beta, batch=batch,
                   stride_a=sa if pad_a else 0, stride_b=sb if pad_b else 0)
    dC = to_device(C0).clone()
    ws = torch.empty(max(plan.workspace_bytes, 16), dtype=torch.uint8, device="cuda")
    plan.run(to_device(A), to_device(B), dC, bias=to_device(bias) if epi else None,
             workspace=ws if plan.workspace_bytes else None, workspace_bytes=plan.workspace_bytes,
             stream=torch.cuda.current_stream().cuda_stream)
    plan.check()
    got = c_to_f64(dC).reshape(M, N)
    c0 = (C0.astype(np.uint32) << 16).view(np.float32) if out_dt == "bf16" else C0
    Y, S = oracle.brgemm(M, N, K, batch, A, B, bias, C0=c0.astype(np.float64).reshape(M, N) if beta else None,
                         in_dtype=oracle.BF16, epilogue=oracle.EPI_BIAS_RELU if epi else oracle.EPI_NONE, beta=float(beta),
                         stride_a=sa, stride_b=sb,
                         layout_a=oracle.BLOCKED32 if layout == "blocked" else oracle.ROW,
                         layout_b=oracle.BLOCKED32 if layout == "blocked" else oracle.TRANSPOSED)
    if integer and out_dt == "f32":
        assert np.array_equal(got, Y), plan.kernel_name
    else:
        tol = TOL_REL_SMAX * S.max() + (TOL_BF16_REL * np.abs(Y) if out_dt == "bf16" else 0.0)
        assert np.all(np.abs(got - Y) <= tol), plan.kernel_name
    return plan


@pytest.mark.parametrize("beta", [0, 1])
def test_listing1_vnni_packed_brgemm_runs_as_printed(beta):
    """The paper's running example (Listing 1): a batch of four 32x32 A tiles and four VNNI-packed 32x192 B tiles
    reduced into one 32x192 C, consumed in the packed layout with no unpacking pass."""
    plan = _run_layout(32, 192, 32, 4, "f32", False, beta, "blocked")
    assert "_br4" in plan.kernel_name and "_bvnni" in plan.kernel_name and "_ablk" in plan.kernel_name
    _run_layout(64, 64, 64, 2, "f32", False, beta, "blocked")          # the appendix BF16 kernel's shape


@pytest.mark.parametrize("mode", ["single", "pair"])
@pytest.mark.parametrize("layout", ["blocked", "transposed"])
@pytest.mark.parametrize("out_dt,epi,beta", [("f32", False, 0), ("f32", True, 1), ("bf16", True, 0)])
def test_brgemm_over_packed_operands(mode, layout, out_dt, epi, beta):
    f = nk.FLAG_SINGLE_CTA if mode == "single" else nk.FLAG_CTA_PAIR
    _run_layout(224, 320, 160, 5, out_dt, epi, beta, layout, pad_a=64, pad_b=32, flags=f)      # gaps between the items
    _run_layout(288, 256, 96, 3, out_dt, epi, beta, layout, flags=f | nk.flag_splitk(2), integer=False, seed=3)
    _run_layout(512, 512, 256, 4, out_dt, epi, beta, layout, integer=False, seed=4)            # plan on auto
