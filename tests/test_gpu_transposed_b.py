"""GPU parity with B kept as its transpose, Bt[N][K] (layout_b = NK_TRANSPOSED): the operand form the tensor
core reads without re-layout (K-major tiles by TMA, like A).  All 16-bit and 8-bit operand types, single CTAs
and pairs, K splits, against the CPU oracle."""
import numpy as np
import pytest
import torch

import nk_inputs
import oracle
import paper_2511_13764_b200 as nk
from nk_testlib import run_and_check

pytestmark = pytest.mark.gpu

INT = ("int", 1.0)
MODES = {"single": nk.FLAG_SINGLE_CTA, "pair": nk.FLAG_CTA_PAIR, "auto": 0}


def W(name, dt, M, N, K, out="f32", epilogue="none", integer=False, seed=1, **kw):
    if integer:
        kw.update(dist_a=INT, dist_b=INT, dist_bias=INT)
    return nk_inputs.Workload(name, M, N, K, dt, out, "b_transposed", epilogue, seed=seed, **kw)


SHAPES = [(128, 64, 128), (100, 72, 160), (1, 8, 16), (130, 200, 416), (384, 328, 1056), (1024, 1024, 1024)]


@pytest.mark.parametrize("dt", ["bf16", "f16", "e4m3", "e5m2"])
@pytest.mark.parametrize("mode,tile", [("single", 2), ("single", 3), ("single", 4), ("pair", 3), ("pair", 4)])
@pytest.mark.parametrize("shape", SHAPES)
def test_bt_exact_on_integer_operands(shape, mode, tile, dt):
    M, N, K = shape
    err, plan = run_and_check(W("bt", dt, M, N, K, integer=True), flags=MODES[mode] | nk.flag_tile_n(tile), exact=True)
    assert "_bt" in plan.kernel_name and "_bvnni" not in plan.kernel_name


@pytest.mark.parametrize("dt,out", [("bf16", "bf16"), ("f16", "f16"), ("e4m3", "f32")])
@pytest.mark.parametrize("mode", ["single", "pair", "auto"])
def test_bt_random_operands_with_epilogue(mode, dt, out):
    run_and_check(W("bt", dt, 200, 328, 272, out, epilogue="bias_relu", seed=5), flags=MODES[mode])
    run_and_check(W("bt", dt, 512, 1024, 2048, out, epilogue="bias_relu", seed=6, dist_a=("normal", 1.0),
                    dist_b=("normal", 0.5)), flags=MODES[mode])


@pytest.mark.parametrize("splits,sep", [(2, False), (4, False), (3, False), (4, True)])
def test_bt_splitk_cluster_and_reduce_kernel(splits, sep):
    f = nk.FLAG_SINGLE_CTA | nk.flag_splitk(splits) | (nk.FLAG_SEPARATE_REDUCE if sep else 0)
    err, plan = run_and_check(W("bt", "bf16", 130, 200, 1104, integer=True), flags=f, exact=True)
    assert ("_cluster" in plan.kernel_name) == (splits in (2, 4) and not sep)
    run_and_check(W("bt", "bf16", 130, 200, 1104, "bf16", epilogue="bias_relu", seed=9), flags=f)


@pytest.mark.parametrize("mode,tile", [("single", 2), ("single", 4), ("pair", 3), ("pair", 4)])
@pytest.mark.parametrize("shape", [(130, 200, 416), (1024, 1024, 1024)])
def test_bt_int8_is_exact(shape, mode, tile):
    M, N, K = shape
    A = nk_inputs.fill(3, nk_inputs.TENSOR_A, M * K, dtype="s8")
    Bt = nk_inputs.fill(3, nk_inputs.TENSOR_B, K * N, dtype="s8")      # read as Bt[N][K]
    plan = nk.Plan(M, N, K, in_dtype=nk.S8, out_dtype=nk.S32, layout_a=nk.ROW_MAJOR, layout_b=nk.TRANSPOSED,
                   flags=MODES[mode] | nk.flag_tile_n(tile) | nk.flag_splitk(1))
    assert plan.kernel_name.endswith("_s8") and "_bt" in plan.kernel_name
    C = torch.full((M * N,), 12345, dtype=torch.int32, device="cuda")
    plan.run(torch.from_numpy(A).cuda(), torch.from_numpy(Bt).cuda(), C, stream=torch.cuda.current_stream().cuda_stream)
    plan.check()
    want = oracle.gemm_s8(M, N, K, A, Bt, layout_b=oracle.TRANSPOSED)
    assert np.array_equal(C.cpu().numpy().astype(np.int64).reshape(M, N), want)


def test_bt_large_shape_sampled_rows():
    w = W("bt", "bf16", 4096, 4096, 4096, seed=12)
    A, B, _ = w.make()
    from nk_testlib import run_plan, check_against_oracle
    got, plan = run_plan(w, A, B, None)
    check_against_oracle(w, got, A, B, None, rows=nk_inputs.stratified_rows(w.seed, w.M, 64))


@pytest.mark.parametrize("dt", ["s8", "e4m3"])
def test_bt_host_buffers_pipelined(dt):
    """nk_gemm_run_host on 8-bit operands large enough for the chunked pipeline (eight row chunks of A, four
    panels of Bt's rows, blocks of C back as they are done): INT8 exactly, E4M3 with its FP32 bias under the
    bound, on 64 stratified rows."""
    M, N, K = 2048, 2048, 2560
    rows = nk_inputs.stratified_rows(31, M, 64)
    if dt == "s8":
        A = nk_inputs.fill(31, nk_inputs.TENSOR_A, M * K, dtype="s8")
        Bt = nk_inputs.fill(31, nk_inputs.TENSOR_B, K * N, dtype="s8")
        bias = None
        plan = nk.Plan(M, N, K, in_dtype=nk.S8, out_dtype=nk.S32, layout_b=nk.TRANSPOSED)
        hC = torch.zeros(M * N, dtype=torch.int32).pin_memory()
    else:
        w = W("bt_host", "e4m3", M, N, K, epilogue="bias_relu", seed=31)
        A, Bt, bias = w.make()
        plan = nk.plan_for(w)
        hC = torch.zeros(M * N, dtype=torch.float32).pin_memory()
    hA, hB = torch.from_numpy(A).pin_memory(), torch.from_numpy(Bt).pin_memory()
    hb = torch.from_numpy(bias).pin_memory() if bias is not None else None
    dA, dB = torch.empty_like(hA, device="cuda"), torch.empty_like(hB, device="cuda")
    db = torch.empty(N, dtype=torch.float32, device="cuda") if bias is not None else None
    dC = torch.empty_like(hC, device="cuda")
    wsb = plan.workspace_bytes
    ws = torch.empty(max(wsb, 16), dtype=torch.uint8, device="cuda")
    for call in range(2):
        hC.fill_(0)
        plan.run_host(hA, hB, hC, dA, dB, dC, hbias=hb, dbias=db, workspace=ws, workspace_bytes=wsb,
                      stream=torch.cuda.current_stream().cuda_stream)
        plan.check()
        got = hC.numpy().reshape(M, N)
        if dt == "s8":
            assert np.array_equal(got[rows].astype(np.int64), oracle.gemm_s8(M, N, K, A, Bt, layout_b=oracle.TRANSPOSED, rows=rows))
        else:
            from nk_testlib import check_against_oracle
            check_against_oracle(w, got.astype(np.float64), A, Bt, bias, rows=rows)


def test_bt_rejects_what_it_cannot_do():
    with pytest.raises(nk.NkError):
        nk.Plan(64, 64, 64, in_dtype=nk.F32, out_dtype=nk.F32, layout_b=nk.TRANSPOSED)
    with pytest.raises(nk.NkError):
        nk.Plan(64, 64, 72, in_dtype=nk.BF16, out_dtype=nk.F32, layout_b=nk.TRANSPOSED)     # K not a multiple of 16
    with pytest.raises(nk.NkError):
        nk.Plan(64, 64, 64, in_dtype=nk.S8, out_dtype=nk.S32, layout_b=nk.TRANSPOSED, batch=2)    # no batch with 8-bit operands
    with pytest.raises(nk.NkError):
        nk.Plan(64, 64, 64, in_dtype=nk.BF16, out_dtype=nk.F32, layout_a=nk.TRANSPOSED)
