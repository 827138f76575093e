"""GPU parity of FP32 operands multiplied on the tensor cores (NK_FLAG_F32_TENSOR): A and B are split
into three BF16 planes each and six cross terms are accumulated in FP32 by the BF16 kernels.  The
paper's FP32 path is FMA arithmetic (Algorithm 1); this variant must meet the same acceptance bound
against the FP64 oracle; for K up to 4096 its error stays under a tenth of that bound."""
import numpy as np
import pytest

import nk_inputs
import paper_2511_13764_b200 as nk
from nk_testlib import run_and_check, run_plan, check_against_oracle

pytestmark = pytest.mark.gpu

INT = ("int", 1.0)
T = nk.FLAG_F32_TENSOR
MODES = {"single": nk.FLAG_SINGLE_CTA, "pair": nk.FLAG_CTA_PAIR, "auto": 0}
FP32_GRADE = 1e-6     # max |c - y| / max sum_k |a.b| (acceptance bound: 1e-5); measured 1.2e-7 .. 3.8e-7, FMA kernels 2e-8 .. 1.2e-7


def W(name, M, N, K, epilogue="none", integer=False, seed=1, **kw):
    if integer:
        kw.update(dist_a=INT, dist_b=INT, dist_bias=INT)
    return nk_inputs.Workload(name, M, N, K, "f32", "f32", "row", epilogue, seed=seed, **kw)


@pytest.mark.parametrize("mode", ["single", "pair", "auto"])
@pytest.mark.parametrize("epi", ["none", "bias_relu"])
def test_integer_operands_are_exact(mode, epi):
    # small integers sit in the hi plane alone: every product and sum is exact, the other five
    # cross terms add zeros, so any mistake in the item -> (A plane, B plane) tables shows
    w = W("f32t_int", 200, 328, 264, epilogue=epi, integer=True)
    err, plan = run_and_check(w, flags=T | MODES[mode], exact=True)
    assert plan.kernel_name.startswith("f32_as_bf16x3_umma_bf16") and "_br6" in plan.kernel_name


@pytest.mark.parametrize("mode", ["single", "pair"])
@pytest.mark.parametrize("shape", [(256, 256, 256), (200, 328, 264), (512, 1024, 2048), (96, 72, 4096)])
def test_fp32_grade_accuracy(shape, mode):
    # uniform and normal operands with full 24-bit significands: all three planes are in use
    M, N, K = shape
    for seed, kw in ((3, {}), (4, dict(dist_a=("normal", 1.0), dist_b=("normal", 0.02)))):
        w = W("f32t", M, N, K, epilogue="bias_relu", seed=seed, **kw)
        err, plan = run_and_check(w, flags=T | MODES[mode])
        assert err < FP32_GRADE, (err, plan.kernel_name)


def test_planes_matter():
    """Against the same operands rounded to BF16 the result differs: the mid and lo planes are used."""
    w = W("f32t", 128, 128, 512, seed=5)
    A, B, _ = w.make()
    c3, _ = run_plan(w, A, B, None, flags=T)
    hi = lambda x: (x.view(np.uint32) & np.uint32(0xFFFF0000)).view(np.float32)
    c1, _ = run_plan(w, hi(A), hi(B), None, flags=T)
    assert not np.array_equal(c3, c1)
    check_against_oracle(w, c3, A, B, None)


@pytest.mark.parametrize("splits,sep", [(2, False), (4, False), (3, False), (4, True)])
@pytest.mark.parametrize("epi", ["none", "bias_relu"])
def test_splitk(splits, sep, epi):
    """K splits of the six-term reduction through the cluster reduction, and through FP32 partials and
    the reduce kernel (which then adds the FP32 bias)."""
    f = T | nk.FLAG_SINGLE_CTA | nk.flag_splitk(splits) | (nk.FLAG_SEPARATE_REDUCE if sep else 0)
    run_and_check(W("f32t_split", 130, 200, 1096, epilogue=epi, integer=True), flags=f, exact=True)
    err, plan = run_and_check(W("f32t_split", 130, 200, 1096, epilogue=epi, seed=9), flags=f)
    assert err < FP32_GRADE


@pytest.mark.parametrize("epi", ["none", "bias_relu"])
def test_tail_wave_split(epi):
    """More 256 x 256 tiles than CTA pairs: the last wave's tiles are cut along the six-term K."""
    w = W("f32t_tail", 2304, 2304, 136, epilogue=epi, seed=11)
    err, plan = run_and_check(w, flags=T | nk.FLAG_CTA_PAIR | nk.flag_tile_n(4) | nk.flag_tail_split(2))
    assert "_tail2" in plan.kernel_name and err < FP32_GRADE


def test_beta_accumulates_into_c():
    w = W("f32t_beta", 160, 136, 264, seed=12)
    A, B, _ = w.make()
    import torch
    from nk_testlib import to_device
    plan = nk.Plan(w.M, w.N, w.K, in_dtype=nk.F32, out_dtype=nk.F32, flags=T, beta=1)
    C0 = nk_inputs.fill(w.seed, nk_inputs.TENSOR_VEC, w.M * w.N, "uniform", 1.0, "f32")
    C = to_device(C0.copy())
    ws = torch.empty(max(plan.workspace_bytes, 16), dtype=torch.uint8, device="cuda:0")
    plan.run(to_device(A), to_device(B), C, workspace=ws, workspace_bytes=plan.workspace_bytes,
             stream=torch.cuda.current_stream().cuda_stream)
    plan.check()
    got = C.cpu().numpy().astype(np.float64).reshape(w.M, w.N) - C0.astype(np.float64).reshape(w.M, w.N)
    check_against_oracle(w, got, A, B, None)


def test_rejects_what_it_cannot_do():
    with pytest.raises(nk.NkError):
        nk.Plan(64, 68, 64, in_dtype=nk.F32, out_dtype=nk.F32, flags=T)          # N not a multiple of 8
    with pytest.raises(nk.NkError):
        nk.Plan(64, 64, 64, in_dtype=nk.F32, out_dtype=nk.F32, flags=T, batch=2)  # batch-reduce
    # the flag means nothing for 16-bit operands
    p = nk.Plan(64, 64, 64, in_dtype=nk.BF16, out_dtype=nk.F32, flags=T)
    assert p.kernel_name.startswith("umma_")
