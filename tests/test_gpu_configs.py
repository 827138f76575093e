"""Full-size parity: the five benchmark configurations, in the launch
configuration bench.py times, against the CPU oracle.

Problems with 2.M.N.K <= 2e10 flop are checked element by element in full.
Larger ones are checked on rows the oracle computes one by one (64 stratified
rows, every 128-row tile band hit; all rows when M <= 128; 4096 seeded columns
when N = 16384) plus a Freivalds identity over the whole of C: C.x = A.(B.x)
for a seeded +-1 vector x, evaluated in float64, which catches a wrong tile
anywhere."""
import functools

import numpy as np
import pytest
import torch

import nk_inputs
import paper_2511_13764_b200 as nk
from nk_testlib import run_plan, check_against_oracle

pytestmark = pytest.mark.gpu


@functools.lru_cache(maxsize=2)
def _cached_fill(seed, tensor, count, dist, sigma, dtype):
    return nk_inputs.fill(seed, tensor, count, dist, sigma, dtype)


def _make(w):
    A = nk_inputs.fill(w.seed, nk_inputs.TENSOR_A, w.M * w.K, w.dist_a[0], w.dist_a[1], w.in_dtype)
    B = _cached_fill(w.seed, nk_inputs.TENSOR_B, w.K * w.N, w.dist_b[0], w.dist_b[1], w.in_dtype)
    bias = None
    if w.epilogue != "none":
        bias = nk_inputs.fill(w.seed, nk_inputs.TENSOR_BIAS, w.N, w.dist_bias[0], w.dist_bias[1], w.in_dtype)
    return A, B, bias


def _as_f64(buf, dtype):
    if dtype == "bf16":
        return (buf.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    if dtype == "f16":
        return buf.view(np.float16).astype(np.float64)
    return buf.astype(np.float64)


def freivalds(w, got, A, B):
    """Row-major, no epilogue: max_i |(C x)_i - (A (B x))_i| against sqrt(N) * 1e-5 * bound."""
    x = np.where(nk_inputs.raw_bits(w.seed, nk_inputs.TENSOR_VEC, 0, w.N) & np.uint64(1), 1.0, -1.0)
    bx = np.empty(w.K)
    absb = np.empty(w.K)
    step = max(1, (1 << 24) // w.N)
    for k0 in range(0, w.K, step):
        blk = _as_f64(B[k0 * w.N:(k0 + step) * w.N], w.in_dtype).reshape(-1, w.N)
        bx[k0:k0 + blk.shape[0]] = blk @ x
        absb[k0:k0 + blk.shape[0]] = np.abs(blk).max(axis=1)
    lhs = got @ x
    rhs = np.empty(w.M)
    bound = np.empty(w.M)
    stepm = max(1, (1 << 24) // w.K)
    for m0 in range(0, w.M, stepm):
        blk = _as_f64(A[m0 * w.K:(m0 + stepm) * w.K], w.in_dtype).reshape(-1, w.K)
        rhs[m0:m0 + blk.shape[0]] = blk @ bx
        bound[m0:m0 + blk.shape[0]] = np.abs(blk) @ absb      # >= any sum_k |a_ik b_kj|
    # Per element the kernel is within 1e-5 * Smax of the exact product (the acceptance bound; `bound` is an
    # upper estimate of Smax).  The row sum over N elements with random signs of x grows like sqrt(N) if the
    # errors are independent; the factor 4 is four standard deviations of that sum, so a correct kernel
    # passes, while one wrong 128-row or 128-column tile (errors of the size of Smax itself) fails by
    # orders of magnitude.
    tol = 4 * np.sqrt(w.N) * 1e-5 * bound.max()
    err = np.abs(lhs - rhs).max()
    assert err <= tol, f"Freivalds check failed: {err} > {tol}"


def check_workload(w, flags=0):
    A, B, bias = _make(w)
    got, plan = run_plan(w, A, B, bias, flags=flags)
    rows = cols = None
    if w.flops > 2e10:
        if w.M > 128:
            rows = nk_inputs.stratified_rows(w.seed, w.M, 64)
        if w.N >= 16384:
            cols = nk_inputs.sample_cols(w.seed, w.N, 4096)
    err = check_against_oracle(w, got, A, B, bias, rows=rows, cols=cols)
    if w.flops > 2e10 and w.layout == "row" and w.epilogue == "none":
        freivalds(w, got, A, B)
    return err, plan


def test_config1_fp32_256():
    err, plan = check_workload(nk_inputs.config(1))
    assert "simt_f32" in plan.kernel_name


def test_config2_bf16_blocked_1024():
    err, plan = check_workload(nk_inputs.config(2))
    assert "umma_bf16" in plan.kernel_name and "_ablk" in plan.kernel_name and "_bvnni" in plan.kernel_name
    check_workload(nk_inputs.config(2), flags=nk.FLAG_REPACK_B)


def test_config3_bf16_mlp_bias_relu():
    err, plan = check_workload(nk_inputs.config(3))
    assert "umma_bf16" in plan.kernel_name


def test_config4_bf16_8192():
    err, plan = check_workload(nk_inputs.config(4))
    assert "umma_bf16_pair_256x256" in plan.kernel_name


@pytest.mark.parametrize("w", nk_inputs.sweep(), ids=lambda w: w.name)
def test_config5_sweep(w):
    check_workload(w)


@pytest.mark.parametrize("w", nk_inputs.paper_mlp(), ids=lambda w: w.name)
def test_paper_mlp_grid(w):
    check_workload(w)


@pytest.mark.parametrize("i", [0, 1, 2])
def test_f16_headline_shapes(i):
    """FP16 operands at full size: 8192^3 on 64 stratified rows plus the Freivalds identity, the two
    MLP layers element by element."""
    w = nk_inputs.f16_set()[i]
    err, plan = check_workload(w)
    assert plan.kernel_name.endswith("_f16")


@pytest.mark.parametrize("name", ["c5_f32_1024x1024x1024", "c5_f32_4096x4096x4096", "c5_f32_128x16384x16384"])
def test_f32_on_tensor_cores_full_size(name):
    """FP32 sweep shapes through the three-plane BF16 split (NK_FLAG_F32_TENSOR): sampled rows against
    the oracle and the Freivalds identity over the whole of C.  The tensor core's FP32 accumulation
    truncates, so the error grows with K: measured 1.0e-6 of max sum |a.b| at K = 16384 (the FMA
    kernels: 2e-8), a fifth of the acceptance bound at worst."""
    w = next(x for x in nk_inputs.sweep() if x.name == name)
    err, plan = check_workload(w, flags=nk.FLAG_F32_TENSOR)
    assert plan.kernel_name.startswith("f32_as_bf16x3_")
    assert err < 2e-6
