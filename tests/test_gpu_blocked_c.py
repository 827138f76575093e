"""Blocked C output ([M/32][N/32][32][32], the layout the next layer reads as its blocked A)
and a multi-layer MLP whose activations never leave the blocked layout (Section 4: packing
happens once, every layer consumes and produces tiles), each layer against the oracle."""
import ctypes

import numpy as np
import pytest
import torch

import nk_inputs
import oracle
import paper_2511_13764_b200 as nk
from nk_testlib import to_device, c_to_f64, TOL_REL_SMAX, TOL_BF16_REL

pytestmark = pytest.mark.gpu


def unblock(flat, M, N):
    """Blocked storage -> logical [M][N]."""
    return flat.reshape(M // 32, N // 32, 32, 32).transpose(0, 2, 1, 3).reshape(M, N)


def test_unblock_matches_the_oracle_index():
    # the oracle's blocked-A index function (an M x N operand) names the same storage order
    M, N = 96, 160
    d = oracle.Desc(M, 32, N, oracle.BF16, oracle.BLOCKED32, oracle.ROW, 0, 0)
    logical = unblock(np.arange(M * N), M, N)
    L = oracle.lib()
    for i, j in [(0, 0), (0, 33), (31, 31), (32, 0), (95, 159), (40, 100), (64, 5)]:
        assert logical[i, j] == L.nko_a_index(ctypes.byref(d), i, j)


def _run(M, N, K, layout, out_dt, epi, beta, flags=0, seed=21):
    w = nk_inputs.Workload("blkc", M, N, K, "bf16", out_dt, layout=layout,
                           epilogue="bias_relu" if epi else "none", seed=seed)
    A, B, bias = w.make()
    C0 = nk_inputs.fill(seed, 5, M * N, "uniform", dtype=out_dt)          # blocked storage of the old C
    lay = nk.BLOCKED32 if layout == "blocked32" else nk.ROW_MAJOR
    plan = nk.Plan(M, N, K, nk.BF16, nk.BF16 if out_dt == "bf16" else nk.F32, layout_a=lay, layout_b=lay,
                   epilogue=nk.EPI_BIAS_RELU if epi else nk.EPI_NONE, flags=flags, beta=beta,
                   layout_c=nk.BLOCKED32)
    assert plan.kernel_name.endswith("_cblk")
    dC = to_device(C0).clone() if beta else torch.full((M * N,), float("nan"), device="cuda",
                                                       dtype=torch.bfloat16 if out_dt == "bf16" else torch.float32)
    ws = torch.empty(max(plan.workspace_bytes, 16), dtype=torch.uint8, device="cuda")
    plan.run(to_device(A), to_device(B), dC, bias=to_device(bias) if epi else None,
             workspace=ws if plan.workspace_bytes else None, workspace_bytes=plan.workspace_bytes,
             stream=torch.cuda.current_stream().cuda_stream)
    plan.check()
    got = unblock(c_to_f64(dC), M, N)
    olay = oracle.BLOCKED32 if layout == "blocked32" else oracle.ROW
    Y, S = oracle.gemm(M, N, K, A, B, None, in_dtype=oracle.BF16, layout_a=olay, layout_b=olay)   # plain product
    if beta:
        c0 = (C0.astype(np.uint32) << 16).view(np.float32) if out_dt == "bf16" else C0
        Y = Y + unblock(c0.astype(np.float64), M, N)
    if epi:
        b = (bias.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
        Y = np.maximum(Y + b[None, :], 0.0)
    assert not np.isnan(got).any()
    tol = TOL_REL_SMAX * (S.max() + 1.0) + (TOL_BF16_REL * np.abs(Y) if out_dt == "bf16" else 0.0)
    bad = np.abs(got - Y) > tol
    assert not bad.any(), (plan.kernel_name, int(bad.sum()), np.argwhere(bad)[:4])
    return plan


@pytest.mark.parametrize("mode", ["single", "pair", "auto"])
@pytest.mark.parametrize("out_dt", ["f32", "bf16"])
@pytest.mark.parametrize("layout", ["row", "blocked32"])
def test_blocked_c(mode, out_dt, layout):
    f = {"single": nk.FLAG_SINGLE_CTA, "pair": nk.FLAG_CTA_PAIR, "auto": 0}[mode]
    _run(288, 352, 160, layout, out_dt, True, 0, flags=f)        # ragged in tiles, whole in blocks
    _run(160, 96, 64, layout, out_dt, False, 1, flags=f)


@pytest.mark.parametrize("out_dt", ["f32", "bf16"])
def test_blocked_c_splitk_and_naive(out_dt):
    p = _run(256, 128, 1024, "row", out_dt, True, 1, flags=nk.FLAG_KERNEL_UMMA | nk.flag_splitk(4))
    assert "splitk4" in p.kernel_name
    _run(64, 96, 64, "blocked32", out_dt, True, 1, flags=nk.FLAG_KERNEL_NAIVE)


def test_mlp_chain_stays_blocked():
    """Three bias+ReLU layers (batch 256; widths 512 -> 1024 -> 768 -> 256): the BF16 output
    of each layer, in blocked storage, is passed as the next layer's blocked A with no
    re-layout in between.  Every layer is checked against the oracle on the very input the
    device used (the previous layer's device output, bit for bit)."""
    batch, widths = 256, [512, 1024, 768, 256]
    seed = 77
    x = to_device(nk_inputs.fill(seed, nk_inputs.TENSOR_A, batch * widths[0], "normal", 1.0, "bf16"))
    ws = torch.empty(64 << 20, dtype=torch.uint8, device="cuda")
    for l in range(3):
        K, N = widths[l], widths[l + 1]
        Wt = nk_inputs.fill(seed + l, nk_inputs.TENSOR_B, K * N, "normal", 0.05, "bf16")    # VNNI-blocked storage
        bias = nk_inputs.fill(seed + l, nk_inputs.TENSOR_BIAS, N, "normal", 0.02, "bf16")
        plan = nk.Plan(batch, N, K, nk.BF16, nk.BF16, layout_a=nk.BLOCKED32, layout_b=nk.BLOCKED32,
                       epilogue=nk.EPI_BIAS_RELU, layout_c=nk.BLOCKED32)
        y = torch.full((batch * N,), float("nan"), dtype=torch.bfloat16, device="cuda")
        assert plan.workspace_bytes <= ws.numel()
        plan.run(x, to_device(Wt), y, bias=to_device(bias), workspace=ws if plan.workspace_bytes else None,
                 workspace_bytes=plan.workspace_bytes, stream=torch.cuda.current_stream().cuda_stream)
        plan.check()
        x_bits = x.cpu().view(torch.int16).numpy().view(np.uint16)
        Y, S = oracle.gemm(batch, N, K, x_bits, Wt, bias, in_dtype=oracle.BF16, layout_a=oracle.BLOCKED32,
                           layout_b=oracle.BLOCKED32, epilogue=oracle.EPI_BIAS_RELU)
        got = unblock(c_to_f64(y), batch, N)
        assert not np.isnan(got).any()
        tol = TOL_REL_SMAX * S.max() + TOL_BF16_REL * np.abs(Y)
        assert np.all(np.abs(got - Y) <= tol), (l, plan.kernel_name)
        assert (got > 0).mean() > 0.2            # the layer is not dead: the next one gets real input
        x = y                                    # blocked C of this layer = blocked A of the next
