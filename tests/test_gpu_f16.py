"""GPU parity of the FP16 operand type (IEEE binary16; Section 5 of the paper names FP16 as the next
packed type): the BF16 kernels with the other 16-bit format, against the CPU oracle."""
import numpy as np
import pytest

import nk_inputs
import paper_2511_13764_b200 as nk
from nk_testlib import run_and_check, run_plan, check_against_oracle

pytestmark = pytest.mark.gpu

INT = ("int", 1.0)
MODES = {"single": nk.FLAG_SINGLE_CTA, "pair": nk.FLAG_CTA_PAIR, "auto": 0}


def W(name, M, N, K, out_dtype="f32", layout="row", epilogue="none", integer=False, seed=1, **kw):
    if integer:
        kw.update(dist_a=INT, dist_b=INT, dist_bias=INT)
    return nk_inputs.Workload(name, M, N, K, "f16", out_dtype, layout, epilogue, seed=seed, **kw)


@pytest.mark.parametrize("mode", ["single", "pair"])
@pytest.mark.parametrize("out_dtype,epi", [("f32", "none"), ("f32", "bias_relu"), ("f16", "none"), ("f16", "bias_relu")])
def test_f16_row_major(out_dtype, epi, mode):
    # integer operands: every product and partial sum is exact, so an FP32 result must equal the oracle
    w = W("f16", 200, 328, 264, out_dtype, epilogue=epi, integer=True)
    err, plan = run_and_check(w, flags=MODES[mode], exact=(out_dtype == "f32"))
    assert plan.kernel_name.endswith("_f16")
    run_and_check(W("f16", 256, 512, 512, out_dtype, epilogue=epi, seed=8), flags=MODES[mode])


def test_f16_differs_from_bf16_on_the_same_bits():
    """The same 16-bit patterns read as BF16 give another product: the format switch reaches the tensor cores."""
    w = W("f16", 128, 128, 128, seed=3)
    A, B, _ = w.make()
    c16, _ = run_plan(w, A, B, None)
    wb = nk_inputs.Workload("bf", 128, 128, 128, "bf16", "f32", seed=3)
    cb, _ = run_plan(wb, A, B, None)
    assert not np.array_equal(c16, cb)
    check_against_oracle(w, c16, A, B, None)


@pytest.mark.parametrize("mode,tile", [("single", 2), ("single", 3), ("pair", 4)])
def test_f16_blocked_vnni(mode, tile):
    w = W("f16blk", 160, 224, 96, layout="blocked32", integer=True)
    err, plan = run_and_check(w, flags=MODES[mode] | nk.flag_tile_n(tile), exact=True)
    assert "_ablk" in plan.kernel_name and "_bvnni" in plan.kernel_name
    run_and_check(W("f16blk", 512, 512, 512, "f16", layout="blocked32", epilogue="bias_relu", seed=10), flags=MODES[mode])


@pytest.mark.parametrize("splits,sep", [(2, False), (4, False), (3, False), (4, True)])
@pytest.mark.parametrize("out_dtype,epi", [("f32", "none"), ("f16", "bias_relu")])
def test_f16_splitk(splits, sep, out_dtype, epi):
    """K splits through the cluster reduction, and through FP32 partials and the reduce kernel."""
    f = nk.FLAG_SINGLE_CTA | nk.flag_splitk(splits) | (nk.FLAG_SEPARATE_REDUCE if sep else 0)
    w = W("f16split", 130, 200, 1096, out_dtype, epilogue=epi, integer=(out_dtype == "f32"))
    err, plan = run_and_check(w, flags=f, exact=(out_dtype == "f32"))
    assert ("_cluster" in plan.kernel_name) == (splits in (2, 4) and not sep)
    run_and_check(W("f16split", 130, 200, 1096, out_dtype, epilogue=epi, seed=9), flags=f)


def test_f16_naive_kernel_and_mlp_shape():
    run_and_check(W("f16naive", 64, 96, 160, "f16", epilogue="bias_relu"), flags=nk.FLAG_KERNEL_NAIVE, expect_kernel="naive")
    # the MLP layer of configuration 3 at a reduced width, FP16 throughout
    w = W("f16mlp", 256, 1024, 1024, "f16", epilogue="bias_relu", dist_a=("normal", 1.0), dist_b=("normal", 0.02), seed=11)
    run_and_check(w)


def test_f16_descriptor_rules():
    with pytest.raises(nk.NkError) as e:
        nk.Plan(128, 128, 128, nk.F16, nk.BF16)      # a 16-bit C has the operands' type
    assert e.value.status == 1
    with pytest.raises(nk.NkError) as e:
        nk.Plan(128, 128, 128, nk.BF16, nk.F16)
    assert e.value.status == 1
    with pytest.raises(nk.NkError) as e:
        nk.Plan(128, 132, 128, nk.F16, nk.F32)       # 16-byte rows, as for BF16
    assert e.value.status == 3
