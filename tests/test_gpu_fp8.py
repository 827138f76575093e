"""GPU parity of 8-bit floating-point operands (E4M3, E5M2): `tcgen05.mma.kind::f8f6f4` with FP32
accumulation, A row-major, B packed in groups of four inside 32 x 32 blocks and re-laid in the kernel,
FP32 bias, FP32 C; against the CPU oracle under the acceptance bound of the 16-bit types."""
import numpy as np
import pytest
import torch

import nk_inputs
import oracle
import paper_2511_13764_b200 as nk
from nk_testlib import run_and_check, run_plan, check_against_oracle

pytestmark = pytest.mark.gpu

INT = ("int", 1.0)
MODES = {"single": nk.FLAG_SINGLE_CTA, "pair": nk.FLAG_CTA_PAIR, "auto": 0}


def W(name, fmt, M, N, K, epilogue="none", integer=False, seed=1, **kw):
    if integer:
        kw.update(dist_a=INT, dist_b=INT, dist_bias=INT)
    return nk_inputs.Workload(name, M, N, K, fmt, "f32", "b_blocked32", epilogue, seed=seed, **kw)


SHAPES = [(128, 64, 128), (100, 96, 160), (1, 32, 32), (130, 160, 416), (384, 320, 1056), (1024, 1024, 1024)]


@pytest.mark.parametrize("fmt", ["e4m3", "e5m2"])
@pytest.mark.parametrize("mode,tile", [("single", 2), ("single", 3), ("single", 4), ("pair", 3), ("pair", 4)])
@pytest.mark.parametrize("shape", SHAPES)
def test_fp8_exact_on_integer_operands(shape, mode, tile, fmt):
    # integers in [-4, 4] are exact in both formats and every partial sum is exact in FP32
    M, N, K = shape
    w = W("fp8", fmt, M, N, K, integer=True)
    err, plan = run_and_check(w, flags=MODES[mode] | nk.flag_tile_n(tile), exact=True)
    assert plan.kernel_name.endswith("_" + fmt) and "_bvnni" in plan.kernel_name


@pytest.mark.parametrize("fmt", ["e4m3", "e5m2"])
@pytest.mark.parametrize("mode", ["single", "pair", "auto"])
@pytest.mark.parametrize("epi", ["none", "bias_relu"])
def test_fp8_random_operands(epi, mode, fmt):
    for M, N, K, kw in ((200, 320, 288, {}), (512, 1024, 2048, dict(dist_a=("normal", 1.0), dist_b=("normal", 0.5)))):
        run_and_check(W("fp8", fmt, M, N, K, epilogue=epi, seed=5, **kw), flags=MODES[mode])


def test_fp8_formats_differ_on_the_same_bits():
    """The same bytes read as E5M2 give another product: the format field reaches the tensor cores."""
    w4 = W("fp8", "e4m3", 128, 128, 128, seed=3)
    A, B, _ = w4.make()
    c4, _ = run_plan(w4, A, B, None)
    w5 = W("fp8", "e5m2", 128, 128, 128, seed=3)
    c5, _ = run_plan(w5, A, B, None)
    assert not np.array_equal(c4, c5)
    check_against_oracle(w4, c4, A, B, None)
    check_against_oracle(w5, c5, A, B, None)


@pytest.mark.parametrize("mode", ["single", "pair"])
@pytest.mark.parametrize("splits,sep", [(2, False), (4, False), (3, False), (4, True)])
@pytest.mark.parametrize("epi", ["none", "bias_relu"])
def test_fp8_splitk_cluster_and_reduce_kernel(splits, sep, epi, mode):
    """K splits inside a thread-block cluster (FP32 pieces through shared memory), and through FP32 partials
    and the reduce kernel; both with the FP32 bias."""
    f = MODES[mode] | nk.flag_splitk(splits) | (nk.FLAG_SEPARATE_REDUCE if sep else 0)
    err, plan = run_and_check(W("fp8", "e4m3", 130, 160, 2080, epilogue=epi, integer=True), flags=f, exact=True)
    assert f"splitk{splits}" in plan.kernel_name
    assert ("_cluster" in plan.kernel_name) == (plan.workspace_bytes == 0)
    if mode == "single":
        assert ("_cluster" in plan.kernel_name) == (splits in (2, 4) and not sep)
    run_and_check(W("fp8", "e5m2", 130, 160, 2080, epilogue=epi, seed=9), flags=f)


def test_fp8_tail_wave_split():
    w = W("fp8", "e4m3", 2304, 2304, 1024, epilogue="bias_relu", seed=11)
    err, plan = run_and_check(w, flags=nk.FLAG_CTA_PAIR | nk.flag_tile_n(4) | nk.flag_tail_split(2))
    assert "_tail2" in plan.kernel_name


@pytest.mark.parametrize("i", [0, 1, 2])
def test_fp8_headline_shapes(i):
    """Full size, plan on auto: 64 stratified rows against the oracle (all columns)."""
    w = nk_inputs.fp8_set()[i]
    A, B, bias = w.make()
    got, plan = run_plan(w, A, B, bias)
    rows = nk_inputs.stratified_rows(w.seed, w.M, 64)
    check_against_oracle(w, got, A, B, bias, rows=rows)


def test_fp8_rejects_what_it_cannot_do():
    ok = dict(in_dtype=nk.E4M3, out_dtype=nk.F32, layout_a=nk.ROW_MAJOR, layout_b=nk.BLOCKED32)
    nk.Plan(64, 64, 64, **ok)
    for bad in (dict(ok, out_dtype=nk.BF16), dict(ok, out_dtype=nk.S32), dict(ok, layout_b=nk.ROW_MAJOR),
                dict(ok, layout_a=nk.BLOCKED32), dict(ok, batch=2), dict(ok, flags=nk.FLAG_KERNEL_NAIVE),
                dict(ok, flags=nk.FLAG_REPACK_B)):
        with pytest.raises(nk.NkError):
            nk.Plan(64, 64, 64, **bad)
    with pytest.raises(nk.NkError):
        nk.Plan(64, 48, 64, **ok)
