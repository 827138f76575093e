"""Shared helpers of the GPU parity tests: upload seeded inputs, run a plan
through the C ABI, compare with the CPU oracle under the acceptance bound."""
from __future__ import annotations

import numpy as np
import torch

import nk_inputs
import oracle
import paper_2511_13764_b200 as nk

TOL_REL_SMAX = 1e-5         # |c - y| <= 1e-5 * max sum_k |a.b|      (FP32 output)
TOL_BF16_REL = 2.0 ** -8    # + 2^-8 * |y| for a BF16-stored output  (one final RNE)
TOL_F16_REL = 2.0 ** -11    # + 2^-11 * |y| for an FP16-stored output (half an ulp of 11 significant bits)
TOL_F16_ABS = 2.0 ** -25    # + half the spacing of FP16 subnormals, for results below 2^-14


def to_device(buf: np.ndarray, device="cuda:0") -> torch.Tensor:
    """16-bit patterns travel as bfloat16 tensors whatever they encode: only the bytes matter."""
    t = torch.from_numpy(buf)
    if buf.dtype == np.uint16:
        t = t.view(torch.bfloat16)
    return t.to(device)


def c_to_f64(C: torch.Tensor) -> np.ndarray:
    if C.dtype == torch.float16:
        return C.cpu().numpy().astype(np.float64)
    if C.dtype == torch.bfloat16:
        bits = C.cpu().view(torch.int16).numpy().view(np.uint16)
        return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    return C.cpu().numpy().astype(np.float64)


def run_plan(w, A, B, bias, flags=0, poison=True, device="cuda:0", plan=None):
    """Returns (C as float64 [M][N], plan).  C is pre-filled with NaN and framed
    by canary bands so that unread/unwritten/overrun elements show up."""
    own = plan is None
    if plan is None:
        plan = nk.plan_for(w, device=torch.device(device).index or 0, flags=flags)
    dA, dB = to_device(A, device), to_device(B, device)
    dbias = to_device(bias, device) if bias is not None else None
    out_dt = {"f32": torch.float32, "bf16": torch.bfloat16, "f16": torch.float16}[w.out_dtype]
    pad = 1024
    Cbuf = torch.full((w.M * w.N + 2 * pad,), float("nan") if poison else 0.0, dtype=out_dt, device=device)
    Cbuf[:pad] = 7.0
    Cbuf[-pad:] = 7.0
    C = Cbuf[pad:pad + w.M * w.N]
    ws_bytes = plan.workspace_bytes
    ws = torch.empty(max(ws_bytes, 16), dtype=torch.uint8, device=device) if ws_bytes else None
    if ws is not None:
        ws.fill_(0xFF)
    plan.run(dA, dB, C, bias=dbias, workspace=ws, workspace_bytes=ws_bytes,
             stream=torch.cuda.current_stream().cuda_stream)
    plan.check()
    torch.cuda.synchronize()
    assert torch.all(Cbuf[:pad] == 7.0) and torch.all(Cbuf[-pad:] == 7.0), "canary overwritten"
    out = c_to_f64(C).reshape(w.M, w.N)
    return out, plan


def describe_mismatch(got, want, bad):
    idx = np.argwhere(bad)
    rows = np.unique(idx[:, 0])
    cols = np.unique(idx[:, 1])
    head = ", ".join(f"({i},{j}): got {got[i, j]:.6g} want {want[i, j]:.6g}" for i, j in idx[:6])
    return (f"{bad.sum()} of {bad.size} elements out of tolerance; rows {rows[:8]}..({len(rows)} distinct), "
            f"cols {cols[:8]}..({len(cols)} distinct); first: {head}")


def check_against_oracle(w, got, A, B, bias, rows=None, cols=None, exact=False):
    """Element-by-element comparison on the rows/cols checked (all by default)."""
    Y, S = oracle.gemm_workload(w, A, B, bias, rows=rows, cols=cols)
    g = got
    if rows is not None:
        g = g[rows, :]
    if cols is not None:
        g = g[:, cols]
    assert not np.isnan(g).any(), f"NaN left in C ({np.isnan(g).sum()} elements never written)"
    if exact:
        bad = g != Y
        assert not bad.any(), describe_mismatch(g, Y, bad)
        return 0.0
    smax = S.max()
    tol = TOL_REL_SMAX * smax
    if w.out_dtype == "bf16":
        tol = tol + TOL_BF16_REL * np.abs(Y)
    if w.out_dtype == "f16":
        tol = tol + TOL_F16_REL * np.abs(Y) + TOL_F16_ABS
    err = np.abs(g - Y)
    bad = err > tol
    assert not bad.any(), describe_mismatch(g, Y, bad) + f" (Smax={smax:.4g})"
    return float(err.max() / smax)


def run_and_check(w, flags=0, exact=False, rows=None, cols=None, expect_kernel=None):
    A, B, bias = w.make()
    got, plan = run_plan(w, A, B, bias, flags=flags)
    if expect_kernel is not None:
        assert expect_kernel in plan.kernel_name, plan.kernel_name
    err = check_against_oracle(w, got, A, B, bias, rows=rows, cols=cols, exact=exact)
    return err, plan
