"""GPU parity: every kernel variant through the C ABI against the CPU oracle.

Small cases use integer-valued operands (exact in FP32 accumulation, so the
comparison is bit-exact and any addressing mistake is unmistakable) and random
operands under the acceptance bound; shapes span several tiles, ragged tails in
M, N and K, and the degenerate sizes (one row, one k-block, K smaller than a
stage)."""
import numpy as np
import pytest
import torch

import nk_inputs
import paper_2511_13764_b200 as nk
from nk_testlib import run_and_check, run_plan, check_against_oracle

pytestmark = pytest.mark.gpu

INT = ("int", 1.0)


def W(name, M, N, K, in_dtype="bf16", out_dtype="f32", layout="row", epilogue="none", integer=False,
      seed=1):
    kw = {}
    if integer:
        kw = dict(dist_a=INT, dist_b=INT, dist_bias=INT)
    return nk_inputs.Workload(name, M, N, K, in_dtype, out_dtype, layout, epilogue, seed=seed, **kw)


# ---------------------------------------------------------------- naive (debug) kernel
@pytest.mark.parametrize("in_dtype,layout,out_dtype,epi", [
    ("f32", "row", "f32", "none"), ("f32", "row", "f32", "bias_relu"),
    ("bf16", "row", "f32", "none"), ("bf16", "blocked32", "f32", "none"),
    ("bf16", "blocked32", "bf16", "bias_relu"),
])
def test_naive_kernel(in_dtype, layout, out_dtype, epi):
    w = W("naive", 64, 96, 160, in_dtype, out_dtype, layout, epi, integer=True)
    run_and_check(w, flags=nk.FLAG_KERNEL_NAIVE, exact=(out_dtype == "f32"), expect_kernel="naive")
    w = W("naive", 64, 96, 160, in_dtype, out_dtype, layout, epi)
    run_and_check(w, flags=nk.FLAG_KERNEL_NAIVE)


# ---------------------------------------------------------------- FP32 SIMT kernel
SIMT_SHAPES = [(256, 256, 256), (1, 4, 4), (33, 132, 68), (128, 128, 16), (130, 260, 100),
               (16, 1024, 1024), (300, 520, 40), (512, 384, 1000)]


@pytest.mark.parametrize("tile", [1, 2, 3])
@pytest.mark.parametrize("shape", SIMT_SHAPES)
def test_simt_f32_exact_integer(shape, tile):
    M, N, K = shape
    w = W("simt", M, N, K, "f32", integer=True)
    run_and_check(w, flags=nk.FLAG_KERNEL_SIMT | nk.flag_tile_n(tile), exact=True, expect_kernel="simt_f32")


SMALL_SHAPES = [(256, 256, 256), (33, 132, 68), (130, 260, 100), (300, 520, 40), (512, 384, 512), (40, 4, 4),
                (64, 64, 8), (900, 320, 36)]


@pytest.mark.parametrize("shape", SMALL_SHAPES)
@pytest.mark.parametrize("epi", ["none", "bias_relu"])
def test_simt_f32_small_kernel(shape, epi):
    """Small FP32 problems (K <= 512, a CTA or two per SM): whole-K slabs in shared memory, four k groups per
    CTA summed in order, one launch, no workspace.  Exact on integer data, then random data; ragged M, N, K."""
    M, N, K = shape
    err, plan = run_and_check(W("small", M, N, K, "f32", epilogue=epi, integer=True), exact=True,
                              expect_kernel="simt_f32_small")
    assert plan.launches_per_run == 1 and plan.workspace_bytes == 0
    run_and_check(W("small", M, N, K, "f32", epilogue=epi, seed=12), expect_kernel="simt_f32_small")


@pytest.mark.parametrize("shape", SIMT_SHAPES)
def test_simt_f32_random_auto(shape):
    M, N, K = shape
    run_and_check(W("simt", M, N, K, "f32", seed=3))


@pytest.mark.parametrize("splits", [2, 5])
@pytest.mark.parametrize("epi", ["none", "bias_relu"])
def test_simt_f32_splitk(splits, epi):
    w = W("simt", 100, 200, 1000, "f32", epilogue=epi, integer=True)
    err, plan = run_and_check(w, flags=nk.flag_splitk(splits) | nk.flag_tile_n(2), exact=True)
    assert f"splitk{splits}" in plan.kernel_name and plan.workspace_bytes >= splits * 100 * 200 * 4
    run_and_check(W("simt", 100, 200, 1000, "f32", epilogue=epi, seed=4), flags=nk.flag_splitk(splits))


def test_simt_f32_bias_relu():
    run_and_check(W("simt", 130, 260, 100, "f32", epilogue="bias_relu", integer=True), exact=True)
    run_and_check(W("simt", 512, 1024, 1024, "f32", epilogue="bias_relu", seed=5))


@pytest.mark.parametrize("epi", ["none", "bias_relu"])
@pytest.mark.parametrize("shape", [(16, 1024, 1024), (1, 4, 4), (7, 520, 100), (32, 2052, 1000),
                                   (17, 512, 64), (16, 4096, 4096)])
def test_simt_f32_skinny(shape, epi):
    """M <= 32 goes to the streaming kernel (one pass over B, K chunks reduced afterwards)."""
    M, N, K = shape
    err, plan = run_and_check(W("skinny", M, N, K, "f32", epilogue=epi, integer=True), exact=True,
                              expect_kernel="simt_f32_skinny")
    run_and_check(W("skinny", M, N, K, "f32", epilogue=epi, seed=6), expect_kernel="simt_f32_skinny")


@pytest.mark.parametrize("splits", [1, 3])
def test_simt_f32_skinny_forced_splits(splits):
    w = W("skinny", 16, 1032, 600, "f32", integer=True)
    err, plan = run_and_check(w, flags=nk.flag_splitk(splits), exact=True, expect_kernel="simt_f32_skinny")
    assert (plan.workspace_bytes > 0) == (plan.launches_per_run == 2)


# ---------------------------------------------------------------- BF16 tcgen05 kernel
UMMA_SHAPES = [(128, 64, 64), (128, 256, 64), (128, 64, 256), (256, 512, 1024), (100, 64, 64),
               (1, 8, 8), (130, 72, 72), (384, 328, 200), (1024, 1024, 1024), (16, 2048, 512)]


MODES = {"single": nk.FLAG_SINGLE_CTA, "pair": nk.FLAG_CTA_PAIR}


def _kernel_prefix(mode, tile):
    bn = 32 << (tile - 1)
    return f"umma_bf16_pair_256x{bn}" if mode == "pair" else f"umma_bf16_128x{bn}"


@pytest.mark.parametrize("mode,tile", [("single", 2), ("single", 3), ("single", 4), ("pair", 3), ("pair", 4)])
@pytest.mark.parametrize("shape", UMMA_SHAPES)
def test_umma_bf16_exact_integer(shape, tile, mode):
    M, N, K = shape
    w = W("umma", M, N, K, "bf16", integer=True)
    run_and_check(w, flags=MODES[mode] | nk.flag_tile_n(tile), exact=True,
                  expect_kernel=_kernel_prefix(mode, tile))


@pytest.mark.parametrize("shape", UMMA_SHAPES)
def test_umma_bf16_random_auto(shape):
    M, N, K = shape
    run_and_check(W("umma", M, N, K, "bf16", seed=7))


@pytest.mark.parametrize("mode", ["single", "pair"])
@pytest.mark.parametrize("out_dtype", ["f32", "bf16"])
@pytest.mark.parametrize("epi", ["none", "bias_relu"])
def test_umma_bf16_epilogues(out_dtype, epi, mode):
    w = W("umma", 200, 328, 264, "bf16", out_dtype, epilogue=epi, integer=(out_dtype == "f32"))
    run_and_check(w, flags=MODES[mode], exact=(out_dtype == "f32"))
    run_and_check(W("umma", 256, 512, 512, "bf16", out_dtype, epilogue=epi, seed=8), flags=MODES[mode])


@pytest.mark.parametrize("mode", ["single", "pair"])
@pytest.mark.parametrize("splits", [2, 3, 7])
@pytest.mark.parametrize("out_dtype,epi", [("f32", "none"), ("bf16", "bias_relu")])
def test_umma_bf16_splitk(splits, out_dtype, epi, mode):
    f = MODES[mode] | nk.flag_splitk(splits)
    w = W("umma", 130, 200, 1096, "bf16", out_dtype, epilogue=epi, integer=(out_dtype == "f32"))
    err, plan = run_and_check(w, flags=f, exact=(out_dtype == "f32"))
    assert "splitk" in plan.kernel_name
    # partials either meet in shared memory (splits = the CTAs of a cluster) or go through the workspace
    assert ("_cluster" in plan.kernel_name) == (plan.workspace_bytes == 0)
    if mode == "single":
        assert ("_cluster" in plan.kernel_name) == (splits in (2, 4, 8))
    assert ("pair" in plan.kernel_name) == (mode == "pair")
    run_and_check(W("umma", 130, 200, 1096, "bf16", out_dtype, epilogue=epi, seed=9), flags=f)


def _cluster_cases():
    """(shape, splits, mode, tile) combinations whose plan forms a cluster: the K splits that survive (no empty
    split) number 2, 4 or 8 (8: single CTAs only), and all the CTAs of the plan are resident at once."""
    out = []
    shapes = [((130, 200, 1096), 2), ((520, 776, 2048), 4), ((256, 1024, 1024), 4), ((16, 1024, 1024), 8),
              ((100, 72, 128), 2), ((300, 520, 512), 2)]
    for (M, N, K), splits in shapes:
        for mode, tile in [("single", 2), ("single", 3), ("single", 4), ("pair", 3), ("pair", 4)]:
            kb = -(-K // 64)
            nsplit = -(-kb // -(-kb // splits))
            bn = 32 << (tile - 1)
            ctas = nsplit * -(-M // (256 if mode == "pair" else 128)) * -(-N // bn) * (2 if mode == "pair" else 1)
            if nsplit in (2, 4) or (nsplit == 8 and mode == "single"):
                if ctas <= 100:
                    out.append(pytest.param((M, N, K), splits, mode, tile, id=f"{M}x{N}x{K}-s{splits}-{mode}-bn{bn}"))
    return out


@pytest.mark.parametrize("out_dtype,epi", [("f32", "none"), ("bf16", "bias_relu")])
@pytest.mark.parametrize("shape,splits,mode,tile", _cluster_cases())
def test_umma_splitk_cluster_reduce_equals_reduce_kernel(shape, splits, out_dtype, epi, mode, tile):
    """K splits as the CTAs (or CTA pairs) of one cluster: the partial sums meet in shared memory and
    are added in split order, exactly as the separate reduce kernel adds them: same bits, one
    launch, no workspace."""
    M, N, K = shape
    w = W("cluster", M, N, K, "bf16", out_dtype, epilogue=epi, seed=21)
    A, B, bias = w.make()
    f = MODES[mode] | nk.flag_splitk(splits) | nk.flag_tile_n(tile)
    c_one, p_one = run_plan(w, A, B, bias, flags=f)
    assert "_cluster" in p_one.kernel_name, p_one.kernel_name
    c_two, p_two = run_plan(w, A, B, bias, flags=f | nk.FLAG_SEPARATE_REDUCE)
    assert p_two.launches_per_run == 2 and p_one.launches_per_run == 1
    assert "_cluster" not in p_two.kernel_name and ("pair" in p_one.kernel_name) == (mode == "pair")
    assert p_one.workspace_bytes == 0 and p_two.workspace_bytes > 0
    assert np.array_equal(c_one, c_two)
    c_again, _ = run_plan(w, A, B, bias, plan=p_one)
    assert np.array_equal(c_again, c_two)
    check_against_oracle(w, c_one, A, B, bias)


@pytest.mark.parametrize("shape,epi,out_dtype", [((256, 4096, 4096), "bias_relu", "bf16"), ((512, 4096, 4096), "bias_relu", "bf16"),
                                                 ((128, 4096, 4096), "none", "f32"), ((512, 1024, 1024), "bias_relu", "bf16")],
                         ids=["c3", "mlp4096", "128rows", "mlp1024"])
def test_cluster_exchange_gives_the_same_bits_every_time(shape, epi, out_dtype):
    """The pieces of a cluster split-K travel as asynchronous remote stores and every receiving warp waits
    on a barrier of its own: whatever order they land in, a full-GPU launch (every SM in some cluster) must
    give the same bits on every one of many back-to-back runs, and those bits are within the bound."""
    M, N, K = shape
    w = W("exchange", M, N, K, "bf16", out_dtype, epilogue=epi, seed=29)
    A, B, bias = w.make()
    first, plan = run_plan(w, A, B, bias)
    assert "_cluster" in plan.kernel_name and plan.launches_per_run == 1, plan.kernel_name
    check_against_oracle(w, first, A, B, bias, rows=nk_inputs.stratified_rows(3, M, 32))
    for _ in range(60):
        again, _ = run_plan(w, A, B, bias, plan=plan)
        assert np.array_equal(again, first)


@pytest.mark.parametrize("mode", ["single", "pair"])
@pytest.mark.parametrize("splits", [2, 4])
def test_umma_splitk_cluster_blocked_operands(splits, mode):
    """Cluster split-K with blocked A, VNNI-blocked B (re-laid in the kernel) and exact integer data."""
    w = W("cluster_blk", 256, 256, 1024, "bf16", layout="blocked32", integer=True)
    err, plan = run_and_check(w, flags=MODES[mode] | nk.flag_splitk(splits) | nk.flag_tile_n(3), exact=True)
    assert "_cluster" in plan.kernel_name and "_bvnni" in plan.kernel_name and plan.workspace_bytes == 0
    assert ("pair" in plan.kernel_name) == (mode == "pair")


@pytest.mark.parametrize("mode,tile", [("single", 2), ("single", 3), ("single", 4), ("pair", 3), ("pair", 4)])
@pytest.mark.parametrize("flags", [0, nk.FLAG_REPACK_B], ids=["inkernel", "repack"])
@pytest.mark.parametrize("shape", [(128, 64, 64), (32, 32, 32), (160, 224, 96), (512, 512, 512)])
def test_umma_bf16_blocked(shape, flags, tile, mode):
    M, N, K = shape
    f = flags | MODES[mode] | nk.flag_tile_n(tile)
    w = W("blk", M, N, K, "bf16", layout="blocked32", integer=True)
    err, plan = run_and_check(w, flags=f, exact=True, expect_kernel=_kernel_prefix(mode, tile))
    assert "_ablk" in plan.kernel_name
    run_and_check(W("blk", M, N, K, "bf16", layout="blocked32", seed=10), flags=f)


def test_blocked_mixed_layouts():
    """A blocked with B row-major, and A row-major with B blocked."""
    import oracle
    M, N, K = 160, 224, 96
    w = W("mix", M, N, K, "bf16", integer=True)
    A, B, _ = w.make()
    for la, lb in ((nk.BLOCKED32, nk.ROW_MAJOR), (nk.ROW_MAJOR, nk.BLOCKED32)):
        plan = nk.Plan(M, N, K, nk.BF16, nk.F32, la, lb)
        got, _ = run_plan(w, A, B, None, plan=plan)
        Y, _ = oracle.gemm(M, N, K, A, B, in_dtype=oracle.BF16, layout_a=la, layout_b=lb)
        assert np.array_equal(got, Y)


def test_repeatable_bit_for_bit():
    w = W("rep", 512, 768, 2048, "bf16", seed=12)
    A, B, bias = w.make()
    c1, plan = run_plan(w, A, B, bias)
    c2, _ = run_plan(w, A, B, bias, plan=plan)
    assert np.array_equal(c1, c2)
    w = W("rep", 256, 256, 512, "f32", seed=13)
    A, B, bias = w.make()
    c1, plan = run_plan(w, A, B, bias, flags=nk.flag_splitk(4))
    c2, _ = run_plan(w, A, B, bias, plan=plan)
    assert np.array_equal(c1, c2)


def test_run_host_entry_point():
    w = W("host", 256, 320, 192, "bf16", "bf16", epilogue="bias_relu", seed=14)
    A, B, bias = w.make()
    plan = nk.plan_for(w)
    hA = torch.from_numpy(A).pin_memory()
    hB = torch.from_numpy(B).pin_memory()
    hb = torch.from_numpy(bias).pin_memory()
    hC = torch.empty(w.M * w.N, dtype=torch.int16).pin_memory()
    dA = torch.empty(A.size, dtype=torch.int16, device="cuda")
    dB = torch.empty(B.size, dtype=torch.int16, device="cuda")
    db = torch.empty(bias.size, dtype=torch.int16, device="cuda")
    dC = torch.empty(w.M * w.N, dtype=torch.int16, device="cuda")
    ws_bytes = plan.workspace_bytes
    ws = torch.empty(max(ws_bytes, 16), dtype=torch.uint8, device="cuda")
    plan.run_host(hA, hB, hC, dA, dB, dC, hbias=hb, dbias=db, workspace=ws, workspace_bytes=ws_bytes,
                  stream=torch.cuda.current_stream().cuda_stream)
    plan.check()
    got = (hC.numpy().view(np.uint16).astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    check_against_oracle(w, got.reshape(w.M, w.N), A, B, bias)


def test_runtime_argument_errors():
    plan = nk.Plan(128, 128, 128, nk.BF16, nk.F32, epilogue=nk.EPI_BIAS_RELU)
    x = torch.zeros(128 * 128, dtype=torch.bfloat16, device="cuda")
    c = torch.zeros(128 * 128, dtype=torch.float32, device="cuda")
    with pytest.raises(nk.NkError) as e:
        plan.run(x, x, c, bias=None)
    assert e.value.status == 1
    with pytest.raises(nk.NkError) as e:
        plan.run(x.data_ptr() + 2, x, c, bias=x)
    assert e.value.status == 3
    plan2 = nk.Plan(128, 128, 1024, nk.BF16, nk.F32, flags=nk.flag_splitk(4) | nk.FLAG_SEPARATE_REDUCE)
    assert plan2.workspace_bytes > 0
    with pytest.raises(nk.NkError) as e:
        plan2.run(x, x, c)
    assert e.value.status == 4


def test_bounded_wait_reports_timeout_and_context_survives():
    """A wait that can never complete gives up after its limit, the kernel exits normally and
    nk_gemm_check reports NK_ERR_TIMEOUT once; the same plan then runs a correct GEMM."""
    w = W("after_timeout", 128, 128, 128, "bf16", integer=True)
    plan = nk.plan_for(w)
    plan.selftest_timeout(stream=torch.cuda.current_stream().cuda_stream)
    with pytest.raises(nk.NkError) as e:
        plan.check()
    assert e.value.status == 7
    plan.check()                                   # the word was cleared
    A, B, bias = w.make()
    got, _ = run_plan(w, A, B, bias, plan=plan)
    check_against_oracle(w, got, A, B, bias, exact=True)


def test_a_timeout_is_reported_by_the_plan_it_happened_in():
    """Every plan has a status word of its own: a wait that ran out in one plan's kernel leaves the
    check of another plan (created before or after it) clean."""
    w = W("whose_timeout", 128, 128, 128, "bf16", integer=True)
    before, plan, after = nk.plan_for(w), nk.plan_for(w), nk.plan_for(w)
    plan.selftest_timeout(stream=torch.cuda.current_stream().cuda_stream)
    before.check()
    after.check()
    with pytest.raises(nk.NkError) as e:
        plan.check()
    assert e.value.status == 7
    plan.check()


@pytest.mark.parametrize("bn", [3, 4])
@pytest.mark.parametrize("out_dtype,epi,splits", [("f32", "none", 2), ("bf16", "bias_relu", 3), ("f32", "bias_relu", 4)])
def test_pair_tail_wave_split(out_dtype, epi, splits, bn):
    """More 256-row tiles than CTA pairs, and a partial last wave: its tiles are cut along K, their FP32
    partials summed by the tail kernel.  Exact integer data, then random data; the plan without the tail
    split gives the same bits when the tail tiles are summed in the same order (two halves of K)."""
    # 10 x 10 (BN = 256) or 10 x 20 (BN = 128) tiles of 256 rows over 74 pairs; ragged M and N
    M, N, K = 2500, 2520, 640
    f = nk.FLAG_CTA_PAIR | nk.flag_tile_n(bn) | nk.flag_splitk(1) | nk.flag_tail_split(splits)
    w = W("tail", M, N, K, "bf16", out_dtype, epilogue=epi, integer=True)
    err, plan = run_and_check(w, flags=f, exact=(out_dtype == "f32"))
    # (equal cuts where the tail tiles times the cuts fit the pairs; else the even share of the k-blocks)
    assert (f"_tail{splits}" in plan.kernel_name or "_streamk" in plan.kernel_name), plan.kernel_name
    assert plan.launches_per_run == 2 and plan.workspace_bytes > 0
    w = W("tail", M, N, K, "bf16", out_dtype, epilogue=epi, seed=31)
    A, B, bias = w.make()
    c_tail, _ = run_plan(w, A, B, bias, flags=f)
    check_against_oracle(w, c_tail, A, B, bias)
    c_plain, p_plain = run_plan(w, A, B, bias, flags=f & ~nk.flag_tail_split(15) | nk.FLAG_NO_TAIL_SPLIT)
    assert "_tail" not in p_plain.kernel_name and "_streamk" not in p_plain.kernel_name
    check_against_oracle(w, c_plain, A, B, bias)


@pytest.mark.parametrize("shape", [(4096, 4096, 704), (3072, 2048, 1088), (2500, 2520, 320)], ids=["3.46waves", "1.3waves", "ragged"])
@pytest.mark.parametrize("out_dtype,epi", [("f32", "none"), ("bf16", "bias_relu")])
def test_pair_stream_k_shares_the_last_wave(shape, out_dtype, epi):
    """More 256 x 256 tiles than CTA pairs and a ragged last wave: the k-blocks of the tiles left over are shared
    out evenly over all the pairs (a pair's range may straddle two tiles), the partial slabs of a tile are
    summed in k order by the tail kernel.  Exact on integer data (bit for bit against the oracle and against
    the plan without the tail treatment), then random data under the acceptance bound."""
    M, N, K = shape
    f = nk.FLAG_CTA_PAIR | nk.flag_tile_n(4) | nk.flag_splitk(1)
    rows = nk_inputs.stratified_rows(5, M, 48)
    w = W("streamk", M, N, K, "bf16", out_dtype, epilogue=epi, integer=True)
    A, B, bias = w.make()
    c_sk, plan = run_plan(w, A, B, bias, flags=f | nk.flag_tail_split(15))
    assert "_streamk" in plan.kernel_name and plan.launches_per_run == 2 and plan.workspace_bytes > 0, plan.kernel_name
    check_against_oracle(w, c_sk, A, B, bias, rows=rows, exact=(out_dtype == "f32"))
    c_plain, p_plain = run_plan(w, A, B, bias, flags=f | nk.FLAG_NO_TAIL_SPLIT)
    assert "_streamk" not in p_plain.kernel_name and "_tail" not in p_plain.kernel_name
    assert np.array_equal(c_sk, c_plain)
    w = W("streamk", M, N, K, "bf16", out_dtype, epilogue=epi, seed=33)
    A, B, bias = w.make()
    c_sk, _ = run_plan(w, A, B, bias, plan=plan)
    check_against_oracle(w, c_sk, A, B, bias, rows=rows)


@pytest.mark.parametrize("layout,K", [("row", 680), ("blocked32", 672)])
def test_pair_k_serpentine_order(layout, K):
    """Three and a half tiles per CTA pair: every other whole tile of a pair is reduced with K walked downwards
    (operand strips shared with the wave before are met where that wave left them in L2).  The order of the sum
    is all that changes: integer data give the oracle's result bit for bit and the same bits as the plan that
    walks K upwards everywhere; random data stay under the acceptance bound, ragged K tail included."""
    M, N = 4096, 4096
    f = nk.FLAG_CTA_PAIR | nk.flag_tile_n(4) | nk.flag_splitk(1) | nk.FLAG_NO_TAIL_SPLIT
    rows = nk_inputs.stratified_rows(9, M, 48)
    w = W("kserp", M, N, K, "bf16", "f32", layout, integer=True, seed=5)
    A, B, bias = w.make()
    c_down, plan = run_plan(w, A, B, bias, flags=f)
    check_against_oracle(w, c_down, A, B, bias, rows=rows, exact=True)
    c_up, _ = run_plan(w, A, B, bias, flags=f | nk.flag_raster(7))
    assert np.array_equal(c_down, c_up)
    w = W("kserp", M, N, K, "bf16", "f32", layout, seed=6)
    A, B, bias = w.make()
    c_down, _ = run_plan(w, A, B, bias, plan=plan)
    check_against_oracle(w, c_down, A, B, bias, rows=rows)
    c_up, _ = run_plan(w, A, B, bias, flags=f | nk.flag_raster(7))
    assert not np.array_equal(c_down, c_up)     # the two orders round differently somewhere: both orders really ran


@pytest.mark.parametrize("out_dtype,bn", [("f32", 4), ("bf16", 4), ("bf16", 3)])
def test_pair_tail_units_follow_tma_stored_tiles(out_dtype, bn):
    """A pair that goes from a whole tile (stored by TMA from its staging tiles) straight to a tail split
    (whose FP32 partial passes through the same staging memory) must first let those stores read their
    source.  Integer data make both plans exact, so the result with the tail split has to equal, bit for
    bit and on every one of many runs, the result of the plan without it."""
    M, N, K = 2500, 2520, 256      # a short K loop: the tail unit's accumulator is ready at once
    w = W("tailrace", M, N, K, "bf16", out_dtype, integer=True, seed=77)
    A, B, bias = w.make()
    f = nk.FLAG_CTA_PAIR | nk.flag_tile_n(bn) | nk.flag_splitk(1)
    c_plain, p_plain = run_plan(w, A, B, bias, flags=f | nk.FLAG_NO_TAIL_SPLIT)
    assert "_tail" not in p_plain.kernel_name
    check_against_oracle(w, c_plain, A, B, bias, exact=(out_dtype == "f32"))
    plan = nk.plan_for(w, flags=f | nk.flag_tail_split(2))
    assert "_tail2" in plan.kernel_name or "_streamk" in plan.kernel_name, plan.kernel_name
    for _ in range(25):
        c_tail, _ = run_plan(w, A, B, bias, plan=plan)
        assert np.array_equal(c_tail, c_plain)


@pytest.mark.parametrize("out_dtype,epi,layout,N", [("f32", "none", "row", 2048), ("bf16", "bias_relu", "row", 2048),
                                                    ("bf16", "bias_relu", "blocked32", 2048), ("f32", "none", "row", 2304)])
def test_run_host_pipelined_chunks(out_dtype, epi, layout, N):
    """Host buffers, a problem large enough for the chunked pipeline (eight row chunks of A, four column
    panels of B when N divides, one otherwise, C back block by block over two copy streams): the result on
    64 stratified rows (every row chunk is hit, all columns) against the oracle, twice."""
    M, K = 2048, 2560
    w = W("hostpipe", M, N, K, "bf16", out_dtype, layout=layout, epilogue=epi, seed=41)
    A, B, bias = w.make()
    plan = nk.plan_for(w)
    odt = torch.float32 if out_dtype == "f32" else torch.int16
    hA, hB = torch.from_numpy(A).pin_memory(), torch.from_numpy(B).pin_memory()
    hb = torch.from_numpy(bias).pin_memory() if bias is not None else None
    hC = torch.empty(M * N, dtype=odt).pin_memory()
    dA = torch.empty(A.size, dtype=torch.int16, device="cuda")
    dB = torch.empty(B.size, dtype=torch.int16, device="cuda")
    db = torch.empty(N, dtype=torch.int16, device="cuda") if bias is not None else None
    dC = torch.empty(M * N, dtype=odt, device="cuda")
    ws_bytes = plan.workspace_bytes
    ws = torch.empty(max(ws_bytes, 16), dtype=torch.uint8, device="cuda")
    rows = nk_inputs.stratified_rows(w.seed, M, 64)
    for call in range(2):
        hC.fill_(0)
        plan.run_host(hA, hB, hC, dA, dB, dC, hbias=hb, dbias=db, workspace=ws, workspace_bytes=ws_bytes,
                      stream=torch.cuda.current_stream().cuda_stream)
        plan.check()
        if out_dtype == "f32":
            got = hC.numpy().astype(np.float64)
        else:
            got = (hC.numpy().view(np.uint16).astype(np.uint32) << 16).view(np.float32).astype(np.float64)
        check_against_oracle(w, got.reshape(M, N), A, B, bias, rows=rows)


# ---------------------------------------------------------------- swap-AB skinny kernel (M <= 64, 16-bit operands)
SWAP_SHAPES = [(16, 1024, 1024), (1, 128, 64), (17, 200, 136), (33, 4096, 512), (64, 328, 1096), (5, 72, 2048),
               (48, 1032, 264)]


@pytest.mark.parametrize("shape", SWAP_SHAPES)
@pytest.mark.parametrize("out_dtype,epi", [("f32", "none"), ("f32", "bias_relu"), ("bf16", "bias_relu")])
def test_swap_ab_skinny_kernel(shape, out_dtype, epi):
    """Few rows of A: B's columns become the rows of the MMA, C leaves transposed back.  Plan on auto (K splits
    inside a cluster where there are several); exact on integer data, then random data; ragged M, N, K."""
    M, N, K = shape
    err, plan = run_and_check(W("swap", M, N, K, "bf16", out_dtype, epilogue=epi, integer=True), exact=(out_dtype == "f32"),
                              expect_kernel="umma_swap")
    assert plan.launches_per_run == 1 and plan.workspace_bytes == 0
    run_and_check(W("swap", M, N, K, "bf16", out_dtype, epilogue=epi, seed=14), expect_kernel="umma_swap")


@pytest.mark.parametrize("splits", [1, 2, 3, 4, 8])
@pytest.mark.parametrize("M", [16, 40, 64])
def test_swap_ab_splits_cluster_equals_reduce_kernel(splits, M):
    """K splits of the skinny kernel: summed in split order inside one CTA of the cluster, or through FP32
    partials and the reduce kernel: the same bits, and both within the bound of the oracle."""
    N, K = 520, 2112
    w = W("swapsplit", M, N, K, "bf16", "f32", epilogue="bias_relu", seed=15)
    A, B, bias = w.make()
    c_one, p_one = run_plan(w, A, B, bias, flags=nk.flag_splitk(splits))
    assert "umma_swap" in p_one.kernel_name and p_one.launches_per_run == 1
    check_against_oracle(w, c_one, A, B, bias)
    if splits > 1 and f"splitk{splits}" in p_one.kernel_name:
        assert "_cluster" in p_one.kernel_name
        c_two, p_two = run_plan(w, A, B, bias, flags=nk.flag_splitk(splits) | nk.FLAG_SEPARATE_REDUCE)
        assert "_cluster" not in p_two.kernel_name and p_two.launches_per_run == 2 and p_two.workspace_bytes > 0
        assert np.array_equal(c_one, c_two)


@pytest.mark.parametrize("dt", ["bf16", "f16"])
@pytest.mark.parametrize("layout", ["row", "b_transposed"])
def test_swap_ab_types_and_transposed_b(dt, layout):
    w = nk_inputs.Workload("swapt", 24, 392 if layout == "row" else 400, 1040, dt, dt, layout, "bias_relu", seed=16,
                           dist_a=("normal", 1.0), dist_b=("uniform", 1.0))
    err, plan = run_and_check(w, expect_kernel="umma_swap")
    assert ("_bt" in plan.kernel_name) == (layout == "b_transposed")
    wi = nk_inputs.Workload("swapt", 24, 384, 1024, dt, "f32", layout, "none", seed=17, dist_a=INT, dist_b=INT)
    run_and_check(wi, exact=True, expect_kernel="umma_swap")
