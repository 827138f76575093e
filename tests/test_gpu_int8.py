"""GPU parity of INT8 operands (the Int8 dot product, Section 5c of the paper; B packed in groups of
four inside 32 x 32 blocks, Section 2): `tcgen05.mma.kind::i8` with INT32 accumulation.  Integer
work: every comparison with the CPU oracle is bit-exact."""
import numpy as np
import pytest
import torch

import nk_inputs
import oracle
import paper_2511_13764_b200 as nk

pytestmark = pytest.mark.gpu

MODES = {"single": nk.FLAG_SINGLE_CTA, "pair": nk.FLAG_CTA_PAIR, "auto": 0}


def run_s8(M, N, K, flags=0, seed=1, A=None, B=None):
    """Returns (C int64 [M][N], plan, A, B-blocked).  C is pre-filled with a canary pattern and framed by bands."""
    if A is None:
        A = nk_inputs.fill(seed, nk_inputs.TENSOR_A, M * K, dtype="s8")
    if B is None:
        B = nk_inputs.fill(seed, nk_inputs.TENSOR_B, K * N, dtype="s8")   # i.i.d. entries: a blocked operand is just a buffer
    plan = nk.Plan(M, N, K, in_dtype=nk.S8, out_dtype=nk.S32, layout_a=nk.ROW_MAJOR, layout_b=nk.BLOCKED32, flags=flags)
    dA, dB = torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda()
    pad = 1024
    Cbuf = torch.full((M * N + 2 * pad,), -(2 ** 31) + 12345, dtype=torch.int32, device="cuda")
    Cbuf[:pad] = 7
    Cbuf[-pad:] = 7
    C = Cbuf[pad:pad + M * N]
    wsb = plan.workspace_bytes            # K splits go through INT32 partials in the workspace
    ws = torch.full((max(wsb, 16),), 0xFF, dtype=torch.uint8, device="cuda")
    plan.run(dA, dB, C, workspace=ws if wsb else None, workspace_bytes=wsb, stream=torch.cuda.current_stream().cuda_stream)
    plan.check()
    torch.cuda.synchronize()
    assert torch.all(Cbuf[:pad] == 7) and torch.all(Cbuf[-pad:] == 7), "canary overwritten"
    return C.cpu().numpy().astype(np.int64).reshape(M, N), plan, A, B


SHAPES = [(128, 64, 128), (128, 256, 32), (100, 96, 160), (1, 32, 32), (130, 160, 416), (384, 320, 1056),
          (1024, 1024, 1024), (16, 2048, 512)]


@pytest.mark.parametrize("mode,tile", [("single", 2), ("single", 3), ("single", 4), ("pair", 3), ("pair", 4)])
@pytest.mark.parametrize("shape", SHAPES)
def test_s8_every_variant_is_exact(shape, mode, tile):
    M, N, K = shape
    got, plan, A, B = run_s8(M, N, K, flags=MODES[mode] | nk.flag_tile_n(tile), seed=3)
    assert plan.kernel_name.endswith("_s8") and "_bvnni" in plan.kernel_name
    assert ("pair" in plan.kernel_name) == (mode == "pair")
    want = oracle.gemm_s8(M, N, K, A, B, layout_b=oracle.BLOCKED32)
    bad = got != want
    assert not bad.any(), f"{bad.sum()} of {bad.size} differ; first at {np.argwhere(bad)[:4].tolist()}"


def test_s8_extreme_values_do_not_overflow():
    """All operands -128: every product is 16384, K = 4096 of them sum to 2^26, far inside INT32."""
    M, N, K = 128, 64, 4096
    A = np.full(M * K, -128, dtype=np.int8)
    B = np.full(K * N, -128, dtype=np.int8)
    got, plan, _, _ = run_s8(M, N, K, A=A, B=B)
    assert np.all(got == 16384 * K)


def test_s8_blocked_b_is_the_packed_flat_matrix():
    """A flat B packed by the oracle's own index rule gives A.B of the flat matrix (numpy, small)."""
    rng = np.random.default_rng(4)
    M, N, K = 64, 96, 160
    A = rng.integers(-128, 128, (M, K), dtype=np.int8)
    Bflat = rng.integers(-128, 128, (K, N), dtype=np.int8)
    got, plan, _, _ = run_s8(M, N, K, A=A.reshape(-1), B=oracle.to_blocked_s8(Bflat))
    assert np.array_equal(got, A.astype(np.int64) @ Bflat.astype(np.int64))


@pytest.mark.parametrize("i", [0, 1, 2])
def test_s8_headline_shapes(i):
    """Full size, the plan left on auto: 64 stratified rows against the oracle (every 128-row band), and an
    exact Freivalds identity over the whole of C: C.x = A.(B.x) in integers for a seeded +-1 vector."""
    w = nk_inputs.s8_set()[i]
    got, plan, A, B = run_s8(w.M, w.N, w.K, seed=w.seed)
    rows = nk_inputs.stratified_rows(w.seed, w.M, 64)
    want = oracle.gemm_s8(w.M, w.N, w.K, A, B, layout_b=oracle.BLOCKED32, rows=rows)
    assert np.array_equal(got[rows], want)
    x = np.where(nk_inputs.raw_bits(w.seed, nk_inputs.TENSOR_VEC, 0, w.N) & np.uint64(1), 1, -1).astype(np.int64)
    # B.x from the blocked storage: [N/32][K/32][8][32][4] -> sum over (n-block, n-in-block)
    Bv = B.reshape(w.N // 32, w.K // 32, 8, 32, 4).astype(np.int64)
    bx = np.einsum("nkqjr,nj->kqr", Bv, x.reshape(w.N // 32, 32)).reshape(w.K)
    lhs = got @ x
    rhs = A.reshape(w.M, w.K).astype(np.int64) @ bx
    assert np.array_equal(lhs, rhs)


@pytest.mark.parametrize("mode", ["single", "pair"])
@pytest.mark.parametrize("splits", [2, 3, 5])
def test_s8_k_splits_add_integer_partials(splits, mode):
    """K splits write INT32 partial sums to the workspace; the reduce kernel adds them as integers: still exact."""
    M, N, K = 130, 160, 2080
    A = nk_inputs.fill(7, nk_inputs.TENSOR_A, M * K, dtype="s8")
    B = nk_inputs.fill(7, nk_inputs.TENSOR_B, K * N, dtype="s8")
    plan = nk.Plan(M, N, K, in_dtype=nk.S8, out_dtype=nk.S32, layout_a=nk.ROW_MAJOR, layout_b=nk.BLOCKED32,
                   flags=MODES[mode] | nk.flag_splitk(splits) | nk.FLAG_SEPARATE_REDUCE)
    assert f"splitk{splits}" in plan.kernel_name and plan.workspace_bytes >= splits * M * N * 4 and plan.launches_per_run == 2
    ws = torch.full((plan.workspace_bytes,), 0xFF, dtype=torch.uint8, device="cuda")
    C = torch.full((M * N,), 12345, dtype=torch.int32, device="cuda")
    plan.run(torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda(), C, workspace=ws, workspace_bytes=plan.workspace_bytes,
             stream=torch.cuda.current_stream().cuda_stream)
    plan.check()
    assert np.array_equal(C.cpu().numpy().astype(np.int64).reshape(M, N), oracle.gemm_s8(M, N, K, A, B, layout_b=oracle.BLOCKED32))


@pytest.mark.parametrize("mode,tile", [("single", 2), ("single", 3), ("single", 4), ("pair", 3), ("pair", 4)])
@pytest.mark.parametrize("splits", [2, 4])
@pytest.mark.parametrize("dequant", [False, True])
def test_s8_k_splits_meet_inside_a_cluster(splits, mode, tile, dequant):
    """K splits as the CTAs (or pairs) of one cluster: the INT32 pieces cross shared memory and are added as
    integers: one launch, no workspace, the exact result; with the dequantising epilogue the FP32 result has
    the bits of the two-kernel path (same integer sum, same FP32 operations after it)."""
    M, N, K = 250, 544, 2080
    A = nk_inputs.fill(17, nk_inputs.TENSOR_A, M * K, dtype="s8")
    B = nk_inputs.fill(17, nk_inputs.TENSOR_B, K * N, dtype="s8")
    bias = nk_inputs.fill(17, nk_inputs.TENSOR_BIAS, N, "normal", 50.0, "f32") if dequant else None
    scale = 1e-4
    sp = torch.cuda.current_stream().cuda_stream
    outs = []
    for extra in (0, nk.FLAG_SEPARATE_REDUCE):
        plan = nk.Plan(M, N, K, in_dtype=nk.S8, out_dtype=nk.F32 if dequant else nk.S32, layout_a=nk.ROW_MAJOR,
                       layout_b=nk.BLOCKED32, epilogue=nk.EPI_BIAS_RELU if dequant else nk.EPI_NONE, scale=scale,
                       flags=MODES[mode] | nk.flag_tile_n(tile) | nk.flag_splitk(splits) | extra)
        assert ("_cluster" in plan.kernel_name) == (extra == 0), plan.kernel_name
        assert (plan.workspace_bytes == 0) == (extra == 0) and plan.launches_per_run == (1 if extra == 0 else 2)
        ws = torch.full((max(plan.workspace_bytes, 16),), 0xFF, dtype=torch.uint8, device="cuda")
        C = torch.full((M * N,), 12345, dtype=torch.float32 if dequant else torch.int32, device="cuda")
        plan.run(torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda(), C, bias=torch.from_numpy(bias).cuda() if dequant else None,
                 workspace=ws if plan.workspace_bytes else None, workspace_bytes=plan.workspace_bytes, stream=sp)
        plan.check()
        outs.append(C.cpu().numpy().reshape(M, N))
    assert np.array_equal(outs[0], outs[1])
    if dequant:
        want, S = oracle.gemm_s8_scaled(M, N, K, A, B, scale, bias=bias, layout_b=oracle.BLOCKED32, relu=True)
        assert np.all(np.abs(outs[0].astype(np.float64) - want) <= DEQ_TOL * S)
    else:
        assert np.array_equal(outs[0].astype(np.int64), oracle.gemm_s8(M, N, K, A, B, layout_b=oracle.BLOCKED32))


@pytest.mark.parametrize("shape", [(4096, 4096, 1408), (3072, 2048, 2176)], ids=["3.46waves", "1.3waves"])
def test_s8_stream_k_is_exact(shape):
    """INT8 operands, a ragged last wave shared out by k-blocks over all the pairs: INT32 partial slabs, added as
    integers by the tail kernel: the exact result on sampled rows, and the same bits as the plan without it."""
    M, N, K = shape
    A = nk_inputs.fill(18, nk_inputs.TENSOR_A, M * K, dtype="s8")
    B = nk_inputs.fill(18, nk_inputs.TENSOR_B, K * N, dtype="s8")
    sp = torch.cuda.current_stream().cuda_stream
    outs = []
    for extra in (nk.flag_tail_split(15), nk.FLAG_NO_TAIL_SPLIT):
        plan = nk.Plan(M, N, K, in_dtype=nk.S8, out_dtype=nk.S32, layout_a=nk.ROW_MAJOR, layout_b=nk.BLOCKED32,
                       flags=nk.FLAG_CTA_PAIR | nk.flag_tile_n(4) | nk.flag_splitk(1) | extra)
        assert ("_streamk" in plan.kernel_name) == (extra != nk.FLAG_NO_TAIL_SPLIT), plan.kernel_name
        ws = torch.full((max(plan.workspace_bytes, 16),), 0xFF, dtype=torch.uint8, device="cuda")
        C = torch.full((M * N,), 12345, dtype=torch.int32, device="cuda")
        plan.run(torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda(), C, workspace=ws if plan.workspace_bytes else None,
                 workspace_bytes=plan.workspace_bytes, stream=sp)
        plan.check()
        outs.append(C.cpu().numpy().reshape(M, N))
    assert np.array_equal(outs[0], outs[1])
    rows = nk_inputs.stratified_rows(18, M, 48)
    assert np.array_equal(outs[0][rows].astype(np.int64), oracle.gemm_s8(M, N, K, A, B, layout_b=oracle.BLOCKED32, rows=rows))


@pytest.mark.parametrize("dequant", [False, True])
def test_s8_tail_wave_split(dequant):
    """More 256 x 256 tiles than CTA pairs: the last wave's tiles are cut along K, their INT32 partials summed
    exactly by the tail reduce kernel (and scaled, biased and rectified there for an FP32 C)."""
    M, N, K = 2304, 2304, 1024
    A = nk_inputs.fill(8, nk_inputs.TENSOR_A, M * K, dtype="s8")
    B = nk_inputs.fill(8, nk_inputs.TENSOR_B, K * N, dtype="s8")
    bias = nk_inputs.fill(8, nk_inputs.TENSOR_BIAS, N, "normal", 50.0, "f32") if dequant else None
    scale = 1e-4
    plan = nk.Plan(M, N, K, in_dtype=nk.S8, out_dtype=nk.F32 if dequant else nk.S32, layout_a=nk.ROW_MAJOR,
                   layout_b=nk.BLOCKED32, epilogue=nk.EPI_BIAS_RELU if dequant else nk.EPI_NONE, scale=scale,
                   flags=nk.FLAG_CTA_PAIR | nk.flag_tile_n(4) | nk.flag_tail_split(2))
    assert "_tail2" in plan.kernel_name
    ws = torch.empty(plan.workspace_bytes, dtype=torch.uint8, device="cuda")
    C = torch.empty(M * N, dtype=torch.float32 if dequant else torch.int32, device="cuda")
    plan.run(torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda(), C, bias=torch.from_numpy(bias).cuda() if dequant else None,
             workspace=ws, workspace_bytes=plan.workspace_bytes, stream=torch.cuda.current_stream().cuda_stream)
    plan.check()
    rows = nk_inputs.stratified_rows(8, M, 96)
    got = C.cpu().numpy().reshape(M, N)[rows]
    if dequant:
        want, S = oracle.gemm_s8_scaled(M, N, K, A, B, scale, bias=bias, layout_b=oracle.BLOCKED32, rows=rows, relu=True)
        assert np.all(np.abs(got.astype(np.float64) - want) <= DEQ_TOL * S)
    else:
        assert np.array_equal(got.astype(np.int64), oracle.gemm_s8(M, N, K, A, B, layout_b=oracle.BLOCKED32, rows=rows))


# ---------------------------------------------------------------- quantised layer: C = scale * (A.B) (+ FP32 bias, ReLU) in FP32
DEQ_TOL = 2.0 ** -22    # int -> FP32, the scaling and the bias add each round once (2^-24 relative each)


@pytest.mark.parametrize("mode,tile", [("single", 2), ("single", 4), ("pair", 3), ("pair", 4), ("auto", 0)])
@pytest.mark.parametrize("epi", ["none", "bias_relu"])
@pytest.mark.parametrize("shape", [(130, 160, 416), (512, 1024, 2048)])
def test_s8_dequantised_output(shape, epi, mode, tile):
    M, N, K = shape
    seed = 5
    A = nk_inputs.fill(seed, nk_inputs.TENSOR_A, M * K, dtype="s8")
    B = nk_inputs.fill(seed, nk_inputs.TENSOR_B, K * N, dtype="s8")
    bias = nk_inputs.fill(seed, nk_inputs.TENSOR_BIAS, N, "normal", 50.0, "f32") if epi != "none" else None
    scale = 0.0123 * 0.0071
    plan = nk.Plan(M, N, K, in_dtype=nk.S8, out_dtype=nk.F32, layout_a=nk.ROW_MAJOR, layout_b=nk.BLOCKED32,
                   epilogue=nk.EPI_BIAS_RELU if bias is not None else nk.EPI_NONE, scale=scale,
                   flags=MODES[mode] | (nk.flag_tile_n(tile) if tile else 0))
    assert plan.kernel_name.endswith("_s8_dequant")
    C = torch.full((M * N,), float("nan"), dtype=torch.float32, device="cuda")
    plan.run(torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda(), C,
             bias=torch.from_numpy(bias).cuda() if bias is not None else None,
             stream=torch.cuda.current_stream().cuda_stream)
    plan.check()
    got = C.cpu().numpy().astype(np.float64).reshape(M, N)
    want, S = oracle.gemm_s8_scaled(M, N, K, A, B, scale, bias=bias, layout_b=oracle.BLOCKED32, relu=bias is not None)
    assert not np.isnan(got).any()
    bad = np.abs(got - want) > DEQ_TOL * S
    assert not bad.any(), f"{bad.sum()} of {bad.size} out of tolerance; first at {np.argwhere(bad)[:4].tolist()}"
    if bias is not None:
        assert (got == 0).any() and (got > 0).any()      # the ReLU is active on part of the output


@pytest.mark.parametrize("n", [1, 3, 4, 7, 1024, 1 << 20, (1 << 20) + 5])
def test_quantize_s8_is_bit_exact(n):
    rng = np.random.default_rng(n)
    x = (rng.standard_normal(n) * 40).astype(np.float32)
    x[: min(n, 8)] = np.array([0.5, 1.5, 2.5, -0.5, 1e9, -1e9, np.nan, -2.5], dtype=np.float32)[: min(n, 8)]
    inv = float(np.float32(1.0 / 0.37))
    dx = torch.from_numpy(x).cuda()
    dq = torch.full((n + 16,), 77, dtype=torch.int8, device="cuda")
    nk.quantize_s8(dx, dq[8:], n, inv, stream=torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    q = dq.cpu().numpy()
    assert np.all(q[:8] == 77) and np.all(q[8 + n:] == 77)
    assert np.array_equal(q[8:8 + n], oracle.quantize_s8(x, inv))


def test_quantised_layer_end_to_end():
    """FP32 activations -> nk_quantize_s8 -> INT8 GEMM with dequantising epilogue, against the oracle fed
    with the oracle's own quantisation of the same activations."""
    M, N, K = 256, 512, 1024
    x = nk_inputs.fill(6, nk_inputs.TENSOR_A, M * K, "normal", 1.0, "f32")
    sx, sw = 4.0 / 127, 0.02
    W8 = nk_inputs.fill(6, nk_inputs.TENSOR_B, K * N, dtype="s8")
    dq = torch.empty(M * K, dtype=torch.int8, device="cuda")
    nk.quantize_s8(torch.from_numpy(x).cuda(), dq, M * K, 1.0 / sx, stream=torch.cuda.current_stream().cuda_stream)
    plan = nk.Plan(M, N, K, in_dtype=nk.S8, out_dtype=nk.F32, layout_a=nk.ROW_MAJOR, layout_b=nk.BLOCKED32, scale=sx * sw)
    C = torch.empty(M * N, dtype=torch.float32, device="cuda")
    plan.run(dq, torch.from_numpy(W8).cuda(), C, stream=torch.cuda.current_stream().cuda_stream)
    plan.check()
    xq = oracle.quantize_s8(x, 1.0 / sx)
    assert np.array_equal(dq.cpu().numpy(), xq)
    want, S = oracle.gemm_s8_scaled(M, N, K, xq, W8, sx * sw, layout_b=oracle.BLOCKED32)
    got = C.cpu().numpy().astype(np.float64).reshape(M, N)
    assert np.all(np.abs(got - want) <= DEQ_TOL * S)


def test_s8_rejects_what_it_cannot_do():
    ok = dict(in_dtype=nk.S8, out_dtype=nk.S32, layout_a=nk.ROW_MAJOR, layout_b=nk.BLOCKED32)
    nk.Plan(64, 64, 64, **ok)
    for bad in (dict(ok, out_dtype=nk.BF16), dict(ok, out_dtype=nk.F32, scale=0.0), dict(ok, layout_b=nk.ROW_MAJOR), dict(ok, layout_a=nk.BLOCKED32),
                dict(ok, epilogue=nk.EPI_BIAS_RELU), dict(ok, beta=1), dict(ok, batch=2),
                dict(ok, flags=nk.FLAG_KERNEL_NAIVE), dict(ok, flags=nk.FLAG_REPACK_B)):
        with pytest.raises(nk.NkError):
            nk.Plan(64, 64, 64, **bad)
    with pytest.raises(nk.NkError):
        nk.Plan(64, 48, 64, **ok)          # N not a multiple of 32
    with pytest.raises(nk.NkError):
        nk.Plan(64, 64, 64, in_dtype=nk.BF16, out_dtype=nk.S32)   # INT32 C belongs to INT8 operands
