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
    assert plan.workspace_bytes == 0
    plan.run(dA, dB, C, stream=torch.cuda.current_stream().cuda_stream)
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


def test_s8_rejects_what_it_cannot_do():
    ok = dict(in_dtype=nk.S8, out_dtype=nk.S32, layout_a=nk.ROW_MAJOR, layout_b=nk.BLOCKED32)
    nk.Plan(64, 64, 64, **ok)
    for bad in (dict(ok, out_dtype=nk.F32), dict(ok, layout_b=nk.ROW_MAJOR), dict(ok, layout_a=nk.BLOCKED32),
                dict(ok, epilogue=nk.EPI_BIAS_RELU), dict(ok, beta=1), dict(ok, batch=2),
                dict(ok, flags=nk.FLAG_KERNEL_NAIVE), dict(ok, flags=nk.FLAG_REPACK_B)):
        with pytest.raises(nk.NkError):
            nk.Plan(64, 64, 64, **bad)
    with pytest.raises(nk.NkError):
        nk.Plan(64, 48, 64, **ok)          # N not a multiple of 32
    with pytest.raises(nk.NkError):
        nk.Plan(64, 64, 64, in_dtype=nk.BF16, out_dtype=nk.S32)   # INT32 C belongs to INT8 operands
    # a forced K split is ignored: INT32 partial sums have no reduce path
    p = nk.Plan(128, 64, 4096, flags=nk.flag_splitk(4), **ok)
    assert "splitk1" in p.kernel_name and p.workspace_bytes == 0
