"""Pins for the CPU oracle: values the paper prints, closed forms, invariants,
brute force in a different loop order, and a library routine on small shapes.
Each is chosen so that a plausible slip in the oracle (dropped term, wrong
index, transposed operand, wrong pair order, missing bias) fails at least one.
"""
import os

import numpy as np
import pytest

import oracle
from oracle import F32, BF16, ROW, BLOCKED32, EPI_NONE, EPI_BIAS_RELU
import nk_inputs

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _bits(x):
    """float array (values exactly representable in BF16) -> uint16 patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    assert np.all((u & 0xFFFF) == 0), "test value is not a BF16 number"
    return (u >> 16).astype(np.uint16)


# ---------------------------------------------------------------- layouts
def test_fig1_vnni2_printed_values():
    flat, packed = [], []
    for line in open(os.path.join(GOLD, "fig1_vnni2.txt")):
        t = line.split()
        if t and t[0] == "flat":
            flat.append([int(v) for v in t[1:]])
        elif t and t[0] == "packed":
            packed.append([int(v) for v in t[1:]])
    flat = np.array(flat, dtype=np.uint16)
    want = np.array(packed, dtype=np.uint16).reshape(2, 4, 2)
    got = oracle.pack_vnni2(flat)
    assert got.shape == (2, 4, 2)
    assert np.array_equal(got, want)
    assert np.array_equal(oracle.unpack_vnni2(got), flat)


def test_vnni2_round_trip_random():
    rng = np.random.default_rng(1)
    x = rng.integers(0, 65536, size=(34, 19), dtype=np.uint16)
    assert np.array_equal(oracle.unpack_vnni2(oracle.pack_vnni2(x)), x)


def test_blocked_b_block_is_fig1_packing_of_the_flat_block():
    """Inside one 32x32 block the blocked-B storage is exactly Figure 1's
    packing of that block; blocks are ordered (n-block, k-block)."""
    K, N = 64, 96
    flat_b = np.arange(K * N, dtype=np.float32).reshape(K, N)
    flat_a = np.zeros((32, K), dtype=np.float32)
    _, Bblk = oracle.to_blocked(flat_a, flat_b, F32)
    Bblk = Bblk.reshape(N // 32, K // 32, 16, 32, 2)
    for nb in range(N // 32):
        for kb in range(K // 32):
            blk = flat_b[kb * 32:(kb + 1) * 32, nb * 32:(nb + 1) * 32]
            want = oracle.pack_vnni2(blk.astype(np.uint16))          # values < 65536
            assert np.array_equal(Bblk[nb, kb].astype(np.uint16), want)


def test_blocked_a_is_block_row_major():
    M, K = 64, 96
    flat_a = np.arange(M * K, dtype=np.float32).reshape(M, K)
    Ablk, _ = oracle.to_blocked(flat_a, np.zeros((K, 32), np.float32), F32)
    Ablk = Ablk.reshape(M // 32, K // 32, 32, 32)
    for mb in range(M // 32):
        for kb in range(K // 32):
            assert np.array_equal(Ablk[mb, kb], flat_a[mb * 32:(mb + 1) * 32, kb * 32:(kb + 1) * 32])


# ---------------------------------------------------------------- bf16 codec
def test_bf16_decode_encode_exhaustive():
    bits = np.arange(65536, dtype=np.uint16)
    exp = (bits >> 7) & 0xFF
    finite = bits[exp != 0xFF]
    f = oracle.bf16_to_f32(finite)
    # decode agrees with the IEEE reading: sign, 8-bit exponent, 7-bit mantissa
    sign = np.where(finite >> 15, -1.0, 1.0)
    e = ((finite >> 7) & 0xFF).astype(np.int64)
    m = (finite & 0x7F).astype(np.float64)
    want = np.where(e == 0, sign * m * 2.0 ** -133, sign * (1 + m / 128) * 2.0 ** (e - 127))
    assert np.array_equal(f.astype(np.float64), want)
    assert np.array_equal(oracle.f32_to_bf16_rne(f), finite)


def test_bf16_rne_ties():
    one = np.float32(1.0)
    cases = [
        (1 + 2.0 ** -8, 1.0),                    # tie, even mantissa -> down
        (1 + 3 * 2.0 ** -8, 1 + 2.0 ** -6),      # tie, odd mantissa -> up
        (1 + 2.0 ** -8 + 2.0 ** -20, 1 + 2.0 ** -7),   # above tie -> up
        (1 + 2.0 ** -8 - 2.0 ** -20, 1.0),       # below tie -> down
        (-(1 + 3 * 2.0 ** -8), -(1 + 2.0 ** -6)),
        (0.0, 0.0),
    ]
    x = np.array([c[0] for c in cases], dtype=np.float32)
    got = oracle.bf16_to_f32(oracle.f32_to_bf16_rne(x))
    assert np.array_equal(got, np.array([c[1] for c in cases], dtype=np.float32))
    assert one == 1.0


def test_input_generator_rounding_matches_oracle_codec():
    v = nk_inputs.fill(3, 0, 5000, "uniform", dtype="f32")
    assert np.array_equal(nk_inputs.f32_to_bf16_bits(v), oracle.f32_to_bf16_rne(v))


# ---------------------------------------------------------------- GEMM core
def _rand_int(shape, seed):
    return np.random.default_rng(seed).integers(-4, 5, size=shape).astype(np.float32)


def test_identity_permutation_diagonal():
    M = K = N = 37
    A = _rand_int((M, K), 2) + np.float32(0.5)
    Y, _ = oracle.gemm(M, N, K, A, np.eye(K, dtype=np.float32))
    assert np.array_equal(Y, A.astype(np.float64))
    perm = np.random.default_rng(3).permutation(K)
    P = np.zeros((K, N), dtype=np.float32)
    P[perm, np.arange(N)] = 1.0                       # (A.P)[:, j] = A[:, perm[j]]
    Y, _ = oracle.gemm(M, N, K, A, P)
    assert np.array_equal(Y, A[:, perm].astype(np.float64))
    Y, _ = oracle.gemm(M, N, K, P, A)                  # (P.A)[i, :] = A[inv[i], :]
    inv = np.argsort(perm)
    assert np.array_equal(Y, A[inv, :].astype(np.float64))
    dvec = (2.0 ** np.random.default_rng(4).integers(-3, 4, size=K)).astype(np.float32)
    Y, _ = oracle.gemm(M, N, K, A, np.diag(dvec))
    assert np.array_equal(Y, (A * dvec[None, :]).astype(np.float64))


def test_rank1_and_all_ones_closed_forms():
    M, N, K = 9, 13, 50
    u = np.arange(-4, 5, dtype=np.float32)
    v = np.arange(-6, 7, dtype=np.float32)
    # K = 1: C = u v^T
    Y, S = oracle.gemm(M, N, 1, u.reshape(M, 1), v.reshape(1, N))
    assert np.array_equal(Y, np.outer(u, v).astype(np.float64))
    assert np.array_equal(S, np.abs(np.outer(u, v)).astype(np.float64))
    # A[i][k] = u_i, B[k][j] = v_j for every k: C = K u v^T
    A = np.repeat(u.reshape(M, 1), K, axis=1)
    B = np.repeat(v.reshape(1, N), K, axis=0)
    Y, S = oracle.gemm(M, N, K, A, B)
    assert np.array_equal(Y, K * np.outer(u, v).astype(np.float64))
    assert np.array_equal(S, K * np.abs(np.outer(u, v)).astype(np.float64))
    Y, _ = oracle.gemm(5, 7, K, np.ones((5, K), np.float32), np.ones((K, 7), np.float32))
    assert np.all(Y == K)


def test_non_square_operand_roles():
    """A is M x K and B is K x N: a transposed or swapped operand changes this result."""
    M, N, K = 3, 5, 7
    A = _rand_int((M, K), 10)
    B = _rand_int((K, N), 11)
    Y, _ = oracle.gemm(M, N, K, A, B)
    want = np.zeros((M, N))
    for j in range(N):                 # j-k-i order: different from the oracle's
        for k in range(K):
            for i in range(M):
                want[i, j] += float(A[i, k]) * float(B[k, j])
    assert np.array_equal(Y, want)


def _shapes():
    for line in open(os.path.join(GOLD, "shapes.txt")):
        if line.startswith("#") or not line.strip():
            continue
        name, batch, M, N, K, dt, lay = line.split()
        yield name, int(batch), int(M), int(N), int(K), dt, lay


@pytest.mark.parametrize("case", list(_shapes()), ids=lambda c: c[0])
def test_paper_example_shapes_brute_force(case):
    """Batch-reduce over the paper's example shapes: sum_i A_i.B_i equals one GEMM
    whose K axis is the concatenation of the batch (Algorithm 1's output line)."""
    name, batch, M, N, K, dt, lay = case
    As = [_rand_int((M, K), 100 + i) for i in range(batch)]
    Bs = [_rand_int((K, N), 200 + i) for i in range(batch)]
    want = np.zeros((M, N))
    for i in range(batch):
        for m in range(M):
            for n in range(N):
                want[m, n] += float(np.dot(As[i][m, :].astype(np.float64), Bs[i][:, n].astype(np.float64)))
    Acat = np.concatenate(As, axis=1)
    Bcat = np.concatenate(Bs, axis=0)
    if dt == "bf16":
        Y, _ = oracle.gemm(M, N, batch * K, _bits(Acat), _bits(Bcat), in_dtype=BF16)
    else:
        Y, _ = oracle.gemm(M, N, batch * K, Acat, Bcat)
    assert np.array_equal(Y, want)
    if lay == "vnni" and M % 32 == 0 and N % 32 == 0:
        Ab, Bb = oracle.to_blocked(_bits(Acat), _bits(Bcat), BF16)
        Yb, _ = oracle.gemm(M, N, batch * K, Ab, Bb, in_dtype=BF16, layout_a=BLOCKED32, layout_b=BLOCKED32)
        assert np.array_equal(Yb, want)


def test_numpy_float64_matmul_small():
    M, N, K = 96, 80, 128
    w = nk_inputs.Workload("t", M, N, K, "f32", "f32", seed=5)
    A, B, _ = w.make()
    Y, S = oracle.gemm_workload(w, A, B, None)
    ref = A.reshape(M, K).astype(np.float64) @ B.reshape(K, N).astype(np.float64)
    sref = np.abs(A.reshape(M, K)).astype(np.float64) @ np.abs(B.reshape(K, N)).astype(np.float64)
    assert np.max(np.abs(Y - ref)) <= 1e-13 * sref.max()
    assert np.max(np.abs(S - sref)) <= 1e-13 * sref.max()


def test_bf16_inputs_decoded_exactly():
    M, N, K = 33, 40, 64
    w = nk_inputs.Workload("t", M, N, K, "bf16", "f32", seed=6)
    A, B, _ = w.make()
    Y, _ = oracle.gemm_workload(w, A, B, None)
    Af = (A.astype(np.uint32) << 16).view(np.float32).reshape(M, K).astype(np.float64)
    Bf = (B.astype(np.uint32) << 16).view(np.float32).reshape(K, N).astype(np.float64)
    assert np.max(np.abs(Y - Af @ Bf)) <= 1e-13 * (np.abs(Af) @ np.abs(Bf)).max()


def test_blocked_equals_flat_bit_for_bit():
    M, N, K = 64, 96, 128
    w = nk_inputs.Workload("t", M, N, K, "bf16", "f32", seed=7)
    A, B, _ = w.make()
    Yf, Sf = oracle.gemm(M, N, K, A, B, in_dtype=BF16)
    Ab, Bb = oracle.to_blocked(A.reshape(M, K), B.reshape(K, N), BF16)
    Yb, Sb = oracle.gemm(M, N, K, Ab, Bb, in_dtype=BF16, layout_a=BLOCKED32, layout_b=BLOCKED32)
    assert np.array_equal(Yf, Yb) and np.array_equal(Sf, Sb)
    # mixed: only B blocked
    Ym, _ = oracle.gemm(M, N, K, A, Bb, in_dtype=BF16, layout_a=ROW, layout_b=BLOCKED32)
    assert np.array_equal(Yf, Ym)


def test_transpose_invariant():
    M, N, K = 17, 23, 31
    A = nk_inputs.fill(8, 0, M * K).reshape(M, K)
    B = nk_inputs.fill(8, 1, K * N).reshape(K, N)
    Y, _ = oracle.gemm(M, N, K, A, B)
    Yt, _ = oracle.gemm(N, M, K, np.ascontiguousarray(B.T), np.ascontiguousarray(A.T))
    assert np.array_equal(Y, Yt.T)     # same products, same k order


def test_row_and_column_subsets_and_thread_independence():
    M, N, K = 50, 60, 70
    A = nk_inputs.fill(9, 0, M * K)
    B = nk_inputs.fill(9, 1, K * N)
    Y, S = oracle.gemm(M, N, K, A, B, nthreads=1)
    Y8, S8 = oracle.gemm(M, N, K, A, B, nthreads=7)
    assert np.array_equal(Y, Y8) and np.array_equal(S, S8)
    rows = np.array([49, 0, 17], dtype=np.int64)
    cols = np.array([3, 59, 4, 30], dtype=np.int64)
    Ys, Ss = oracle.gemm(M, N, K, A, B, rows=rows, cols=cols)
    assert np.array_equal(Ys, Y[np.ix_(rows, cols)])
    assert np.array_equal(Ss, S[np.ix_(rows, cols)])


# ---------------------------------------------------------------- epilogue
def test_epilogue_closed_forms():
    M, N, K = 12, 20, 16
    A = _rand_int((M, K), 20)
    B = _rand_int((K, N), 21)
    C = A.astype(np.float64) @ B.astype(np.float64)
    big = np.full(N, 1024.0, dtype=np.float32)
    Y, S = oracle.gemm(M, N, K, A, B, big, epilogue=EPI_BIAS_RELU)
    assert np.array_equal(Y, C + 1024.0)              # ReLU inactive: GEMM + bias
    _, S0 = oracle.gemm(M, N, K, A, B)
    assert np.array_equal(S, S0 + 1024.0)             # |bias| enters the scale
    Y, _ = oracle.gemm(M, N, K, A, B, -big, epilogue=EPI_BIAS_RELU)
    assert np.all(Y == 0.0)                           # everything clipped
    # per-column bias: column j shifted by j - 8, clipped at zero
    bias = (np.arange(N) - 8).astype(np.float32)
    Y, _ = oracle.gemm(M, N, K, A, B, bias, epilogue=EPI_BIAS_RELU)
    assert np.array_equal(Y, np.maximum(C + bias[None, :].astype(np.float64), 0.0))
    # bias = -(row of A.B) on a one-row problem: exactly zero
    Y, _ = oracle.gemm(1, N, K, A[:1], B, (-C[0]).astype(np.float32), epilogue=EPI_BIAS_RELU)
    assert np.all(Y == 0.0)
    with pytest.raises(ValueError):
        oracle.gemm(M, N, K, A, B, None, epilogue=EPI_BIAS_RELU)


def test_bf16_bias_decoded():
    M, N, K = 4, 8, 8
    A = _bits(_rand_int((M, K), 30))
    B = _bits(_rand_int((K, N), 31))
    bias = _bits(np.full(N, 0.5, dtype=np.float32))
    Y, _ = oracle.gemm(M, N, K, A, B, bias, in_dtype=BF16, epilogue=EPI_BIAS_RELU)
    Y0, _ = oracle.gemm(M, N, K, A, B, in_dtype=BF16)
    assert np.array_equal(Y, np.maximum(Y0 + 0.5, 0.0))


# ---------------------------------------------------------------- tolerance sanity
def test_fp32_sequential_accumulation_meets_the_bar():
    """The acceptance bar (1e-5 x max sum|a.b|) is reachable by FP32 accumulation:
    the oracle's own FP32-sequential mode passes it at K = 16384."""
    M, N, K = 4, 64, 16384
    w = nk_inputs.Workload("t", M, N, K, "bf16", "f32", seed=11)
    A, B, _ = w.make()
    Y, S = oracle.gemm_workload(w, A, B, None)
    Y32, _ = oracle.gemm_workload(w, A, B, None, acc_mode=oracle.ACC_F32_SEQ)
    err = np.max(np.abs(Y - Y32)) / S.max()
    assert 0 < err <= 1e-5


def test_planted_mistakes_are_caught():
    """A wrong VNNI pair order or a dropped k term changes results the pins fix."""
    flat = np.arange(16, dtype=np.uint16).reshape(4, 4)
    good = oracle.pack_vnni2(flat)
    swapped = good[:, :, ::-1]
    assert not np.array_equal(swapped, good)
    M, N, K = 4, 4, 8
    A = _rand_int((M, K), 40) + 1
    B = _rand_int((K, N), 41) + 1
    Y, _ = oracle.gemm(M, N, K, A, B)
    Ydrop, _ = oracle.gemm(M, N, K - 1, np.ascontiguousarray(A[:, :-1]), np.ascontiguousarray(B[:-1]))
    assert not np.array_equal(Y, Ydrop)


# ---------------------------------------------------------------- generator
def test_generator_golden_and_ranges():
    """SplitMix64's published test vector (seed 1234567: first outputs) pins mix64;
    ranges and grid of the uniform draw; normal moments."""
    # SplitMix64 state s -> output mix64(s + GOLDEN); known vector for seed 1234567
    s = np.array([1234567], dtype=np.uint64)
    with np.errstate(over="ignore"):
        o1 = nk_inputs.mix64(s + nk_inputs.GOLDEN)[0]
        o2 = nk_inputs.mix64(s + nk_inputs.GOLDEN * np.uint64(2))[0]
    assert int(o1) == 6457827717110365317 and int(o2) == 3203168211198807973
    u = nk_inputs.fill(1, 0, 200000)
    assert u.min() >= -1.0 and u.max() < 1.0
    assert np.all(u * 2.0 ** 23 == np.round(u * 2.0 ** 23))
    assert abs(u.mean()) < 0.01 and abs(u.var() - 1 / 3) < 0.01
    z = nk_inputs.fill(1, 1, 200000, "normal", 0.02)
    assert abs(z.mean()) < 3e-4 and abs(z.std() - 0.02) < 3e-4
    # stateless: any slice equals the same indices of a longer buffer
    assert np.array_equal(nk_inputs.fill(1, 0, 100), u[:100])
    rows = nk_inputs.stratified_rows(4017, 8192, 64)
    assert len(rows) == 64 and np.array_equal(rows // 128, np.arange(64))


# ---------------------------------------------------------------- batch-reduce GEMM, beta
@pytest.mark.parametrize("case", list(_shapes()), ids=lambda c: c[0])
def test_brgemm_paper_shapes_against_k_concatenation(case):
    """sum_b A_b.B_b over the paper's example shapes, through the batch interface, equals the
    plain GEMM on K-concatenated operands bit for bit (same products, same order) and a
    brute-force sum written in another loop order."""
    name, batch, M, N, K, dt, lay = case
    As = [_rand_int((M, K), 300 + i) for i in range(batch)]
    Bs = [_rand_int((K, N), 400 + i) for i in range(batch)]
    A = np.stack(As).reshape(-1)
    B = np.stack(Bs).reshape(-1)
    if dt == "bf16":
        Y, S = oracle.brgemm(M, N, K, batch, _bits(A), _bits(B), in_dtype=BF16)
        Yc, Sc = oracle.gemm(M, N, batch * K, _bits(np.concatenate(As, axis=1)), _bits(np.concatenate(Bs, axis=0)),
                             in_dtype=BF16)
    else:
        Y, S = oracle.brgemm(M, N, K, batch, A, B)
        Yc, Sc = oracle.gemm(M, N, batch * K, np.concatenate(As, axis=1), np.concatenate(Bs, axis=0))
    assert np.array_equal(Y, Yc) and np.array_equal(S, Sc)
    want = np.zeros((M, N))
    for n in range(N):
        for b in reversed(range(batch)):
            want[:, n] += As[b].astype(np.float64) @ Bs[b][:, n].astype(np.float64)
    assert np.array_equal(Y, want)          # integers: exact in any order


def test_brgemm_beta_and_strides():
    M, N, K, batch = 5, 7, 6, 3
    sa, sb = M * K + 11, K * N + 5                      # non-contiguous batch items
    rng = np.random.default_rng(50)
    A = rng.integers(-4, 5, size=(batch - 1) * sa + M * K).astype(np.float32)
    B = rng.integers(-4, 5, size=(batch - 1) * sb + K * N).astype(np.float32)
    ref = np.zeros((M, N))
    for b in range(batch):
        ref += A[b * sa:b * sa + M * K].reshape(M, K).astype(np.float64) @ \
               B[b * sb:b * sb + K * N].reshape(K, N).astype(np.float64)
    Y, _ = oracle.brgemm(M, N, K, batch, A, B, stride_a=sa, stride_b=sb)
    assert np.array_equal(Y, ref)
    C0 = rng.integers(-9, 10, size=(M, N)).astype(np.float64)
    Y1, S1 = oracle.brgemm(M, N, K, batch, A, B, C0=C0, beta=1.0, stride_a=sa, stride_b=sb)
    assert np.array_equal(Y1, ref + C0)                 # beta = 1 adds the old C
    Y0, S0 = oracle.brgemm(M, N, K, batch, A, B, C0=C0, beta=0.0, stride_a=sa, stride_b=sb)
    assert np.array_equal(Y0, ref)                      # beta = 0 ignores it
    assert np.array_equal(S1, S0 + np.abs(C0))
    Yz, _ = oracle.brgemm(M, N, K, batch, A, B, C0=-ref, beta=1.0, stride_a=sa, stride_b=sb)
    assert np.all(Yz == 0.0)                            # C0 = -(sum) cancels exactly
    Ya, _ = oracle.brgemm(M, N, K, batch, np.zeros_like(A), B, C0=C0, beta=1.0, stride_a=sa, stride_b=sb)
    assert np.array_equal(Ya, C0)                       # zero A leaves C0
    bias = np.full(N, -1000.0, dtype=np.float32)
    Yr, _ = oracle.brgemm(M, N, K, batch, A, B, bias, C0=C0, beta=1.0, epilogue=EPI_BIAS_RELU, stride_a=sa, stride_b=sb)
    assert np.all(Yr == 0.0)
    with pytest.raises(ValueError):
        oracle.brgemm(M, N, K, batch, A, B, beta=1.0, stride_a=sa, stride_b=sb)      # beta = 1 needs C0
    with pytest.raises(ValueError):
        oracle.brgemm(M, N, K, batch, A, B, C0=C0, beta=0.5, stride_a=sa, stride_b=sb)


def _pack_items_figure1(As, Bs):
    """Blocked storage of batch items written with numpy reshapes from the layout's definition (not with the
    oracle's index functions): A[M/32][K/32][32][32]; B[N/32][K/32][16][32][2] with Figure 1's rule
    packed[k/2][n][k%2] = flat[k][n] inside every 32 x 32 block."""
    out_a, out_b = [], []
    for A, B in zip(As, Bs):
        M, K = A.shape
        N = B.shape[1]
        out_a.append(A.reshape(M // 32, 32, K // 32, 32).transpose(0, 2, 1, 3).reshape(-1))
        blk = B.reshape(K // 32, 32, N // 32, 32).transpose(2, 0, 1, 3)          # [n-block][k-block][k][n]
        out_b.append(blk.reshape(N // 32, K // 32, 16, 2, 32).transpose(0, 1, 2, 4, 3).reshape(-1))
    return out_a, out_b


@pytest.mark.parametrize("M,N,K,batch", [(32, 192, 32, 4), (64, 64, 64, 2), (96, 32, 160, 3)])
def test_brgemm_over_blocked_items_is_the_flat_brgemm(M, N, K, batch):
    """Listing 1's kernel is a batch-reduce over VNNI-packed items.  Items packed from the layout's definition
    (numpy reshapes, Figure 1's pair rule) give, through the blocked interface, bit for bit what the flat
    interface gives on the flat items (same products, same k order), also with gaps between the items and
    with beta = 1; a swapped pair order or a transposed block is caught."""
    As = [_rand_int((M, K), 700 + i) for i in range(batch)]
    Bs = [_rand_int((K, N), 800 + i) for i in range(batch)]
    Yf, Sf = oracle.brgemm(M, N, K, batch, _bits(np.stack(As).reshape(-1)), _bits(np.stack(Bs).reshape(-1)), in_dtype=BF16)
    pa, pb = _pack_items_figure1(As, Bs)
    gap_a, gap_b = 64, 32
    A = np.zeros((batch - 1) * (M * K + gap_a) + M * K, dtype=np.float32)
    B = np.zeros((batch - 1) * (K * N + gap_b) + K * N, dtype=np.float32)
    for b in range(batch):
        A[b * (M * K + gap_a):b * (M * K + gap_a) + M * K] = pa[b]
        B[b * (K * N + gap_b):b * (K * N + gap_b) + K * N] = pb[b]
    kw = dict(in_dtype=BF16, layout_a=BLOCKED32, layout_b=BLOCKED32, stride_a=M * K + gap_a, stride_b=K * N + gap_b)
    Yb, Sb = oracle.brgemm(M, N, K, batch, _bits(A), _bits(B), **kw)
    assert np.array_equal(Yb, Yf) and np.array_equal(Sb, Sf)
    C0 = _rand_int((M, N), 900).astype(np.float64)
    Y1, _ = oracle.brgemm(M, N, K, batch, _bits(A), _bits(B), C0=C0, beta=1.0, **kw)
    assert np.array_equal(Y1, Yf + C0)
    # planted mistakes: the odd/even pair swapped inside B's words; B's block read as its transpose
    Bsw = B.copy()
    for b in range(batch):
        seg = Bsw[b * (K * N + gap_b):b * (K * N + gap_b) + K * N].reshape(-1, 2)
        seg[:] = seg[:, ::-1]
    Yw, _ = oracle.brgemm(M, N, K, batch, _bits(A), _bits(Bsw), **kw)
    assert not np.array_equal(Yw, Yf)
    # mixed forms: blocked A with flat B, flat A with blocked B
    Ym, _ = oracle.brgemm(M, N, K, batch, _bits(A), _bits(np.stack(Bs).reshape(-1)), in_dtype=BF16, layout_a=BLOCKED32,
                          stride_a=M * K + gap_a)
    assert np.array_equal(Ym, Yf)
    Yn, _ = oracle.brgemm(M, N, K, batch, _bits(np.stack(As).reshape(-1)), _bits(B), in_dtype=BF16, layout_b=BLOCKED32,
                          stride_b=K * N + gap_b)
    assert np.array_equal(Yn, Yf)


def test_brgemm_batch_one_is_gemm():
    M, N, K = 9, 12, 20
    A = nk_inputs.fill(60, 0, M * K)
    B = nk_inputs.fill(60, 1, K * N)
    Y, S = oracle.brgemm(M, N, K, 1, A, B)
    Yg, Sg = oracle.gemm(M, N, K, A, B)
    assert np.array_equal(Y, Yg) and np.array_equal(S, Sg)


# ---------------------------------------------------------------- FP16 operands (Section 5: the next packed type)
def test_f16_decode_exhaustive_against_ieee_and_numpy():
    bits = np.arange(65536, dtype=np.uint16)
    e = ((bits >> 10) & 0x1F).astype(np.int64)
    finite = bits[e != 31]
    f = oracle.f16_to_f32(finite).astype(np.float64)
    ef = ((finite >> 10) & 0x1F).astype(np.int64)
    m = (finite & 0x3FF).astype(np.float64)
    sign = np.where(finite >> 15, -1.0, 1.0)
    want = np.where(ef == 0, sign * m * 2.0 ** -24, sign * (1 + m / 1024) * 2.0 ** (ef - 15))
    assert np.array_equal(f, want)
    # the same through the library's binary16 type (a separate implementation of the format)
    assert np.array_equal(f, finite.view(np.float16).astype(np.float64))
    # landmarks of the format: 1, -2, the smallest subnormal, the largest finite value, 1/3 rounded
    marks = np.array([0x3C00, 0xC000, 0x0001, 0x7BFF, 0x3555], dtype=np.uint16)
    assert np.array_equal(oracle.f16_to_f32(marks).astype(np.float64),
                          np.array([1.0, -2.0, 2.0 ** -24, 65504.0, 1365 / 4096]))
    inf = oracle.f16_to_f32(np.array([0x7C00, 0xFC00], dtype=np.uint16))
    assert np.isposinf(inf[0]) and np.isneginf(inf[1])


def test_f16_generator_rounds_to_nearest_even():
    v = nk_inputs.fill(4, 0, 20000, "uniform", dtype="f32")
    h = nk_inputs.f32_to_f16_bits(v)
    back = oracle.f16_to_f32(h).astype(np.float64)
    x = v.astype(np.float64)
    ulp = np.where(np.abs(back) >= 2.0 ** -14, 2.0 ** (np.floor(np.log2(np.maximum(np.abs(back), 2.0 ** -14))) - 10), 2.0 ** -24)
    assert np.all(np.abs(back - x) <= ulp / 2 * (1 + 1e-12))
    ties = np.array([1 + 2.0 ** -11, 1 + 3 * 2.0 ** -11, -(1 + 3 * 2.0 ** -11), 1 + 2.0 ** -11 + 2.0 ** -20], dtype=np.float32)
    got = oracle.f16_to_f32(nk_inputs.f32_to_f16_bits(ties)).astype(np.float64)
    assert np.array_equal(got, np.array([1.0, 1 + 2.0 ** -9, -(1 + 2.0 ** -9), 1 + 2.0 ** -10]))
    assert np.array_equal(nk_inputs.fill(4, 0, 100, "uniform", dtype="f16"), nk_inputs.f32_to_f16_bits(v[:100]))


def test_f16_gemm_equals_gemm_of_the_widened_operands():
    """FP16 operands, row-major and blocked, with bias: the oracle on the 16-bit storage equals, bit
    for bit, the oracle on the same values stored as FP32 (widening is exact, the order is the same)."""
    M, N, K = 64, 96, 128
    for layout in ("row", "blocked32"):
        w = nk_inputs.Workload("t", M, N, K, "f16", "f32", layout=layout, epilogue="bias_relu", seed=9)
        A, B, bias = w.make()
        Y, S = oracle.gemm_workload(w, A, B, bias)
        widen = lambda x: x.view(np.float16).astype(np.float32)
        lay = BLOCKED32 if layout == "blocked32" else ROW
        if layout == "blocked32":
            # blocked storage of FP32 is not a product layout, but the oracle's index functions do not care
            Y2, S2 = oracle.gemm(M, N, K, widen(A), widen(B), widen(bias), in_dtype=F32, layout_a=lay, layout_b=lay,
                                 epilogue=EPI_BIAS_RELU)
        else:
            Y2, S2 = oracle.gemm(M, N, K, widen(A), widen(B), widen(bias), in_dtype=F32, epilogue=EPI_BIAS_RELU)
        assert np.array_equal(Y, Y2) and np.array_equal(S, S2)
    # integer data: exact closed form through numpy
    w = nk_inputs.Workload("t", 40, 48, 64, "f16", "f32", dist_a=("int", 1.0), dist_b=("int", 1.0), seed=10)
    A, B, _ = w.make()
    Y, _ = oracle.gemm_workload(w, A, B, None)
    Af = A.view(np.float16).astype(np.float64).reshape(40, 64)
    Bf = B.view(np.float16).astype(np.float64).reshape(64, 48)
    assert np.array_equal(Y, Af @ Bf)
    # a BF16 reading of the same bits gives something else: the dtype switch is live
    Yb, _ = oracle.gemm(40, 48, 64, A, B, in_dtype=BF16)
    assert not np.array_equal(Y, Yb)


# ---------------------------------------------------------------- INT8 (Section 5c; packing in groups of four, Section 2)
def test_vnni4_is_fig1_rule_with_groups_of_four():
    """Figure 1's flat 4 x 4 matrix 0..15 under the same rule with four k per group: one row of
    quadruples (0,4,8,12) (1,5,9,13) (2,6,10,14) (3,7,11,15); and the pair packing of Figure 1 is what
    the quadruple packing gives when rows 2k, 2k+1 are read out of a quadruple's halves."""
    flat = np.arange(16, dtype=np.int8).reshape(4, 4)
    p4 = oracle.pack_vnni4(flat)
    assert p4.tolist() == [[[0, 4, 8, 12], [1, 5, 9, 13], [2, 6, 10, 14], [3, 7, 11, 15]]]
    with open(os.path.join(GOLD, "fig1_vnni2.txt")) as f:
        printed = [[int(v) for v in line.split()[1:]] for line in f if line.startswith("packed")]
    halves = [[v for q in p4[0].tolist() for v in q[0:2]], [v for q in p4[0].tolist() for v in q[2:4]]]
    assert halves == printed
    rng = np.random.default_rng(5)
    x = rng.integers(-128, 128, (64, 96), dtype=np.int8)
    assert np.array_equal(oracle.unpack_vnni4(oracle.pack_vnni4(x)), x)


def test_s8_blocked_b_block_is_vnni4_packing_of_the_flat_block():
    rng = np.random.default_rng(6)
    K, N = 64, 96
    flat = rng.integers(-128, 128, (K, N), dtype=np.int8)
    blk = oracle.to_blocked_s8(flat).reshape(N // 32, K // 32, 8, 32, 4)
    for nb in range(N // 32):
        for kb in range(K // 32):
            want = oracle.pack_vnni4(flat[kb * 32:(kb + 1) * 32, nb * 32:(nb + 1) * 32])
            assert np.array_equal(blk[nb, kb], want)


def test_s8_gemm_closed_forms_and_numpy():
    rng = np.random.default_rng(7)
    M, N, K = 37, 64, 96
    A = rng.integers(-128, 128, (M, K), dtype=np.int8)
    B = rng.integers(-128, 128, (K, N), dtype=np.int8)
    want = A.astype(np.int64) @ B.astype(np.int64)            # library routine on a small case
    got = oracle.gemm_s8(M, N, K, A, B)
    assert got.dtype == np.int64 and np.array_equal(got, want)
    # blocked B gives the same integers; so does any row subset and any thread count
    Bb = oracle.to_blocked_s8(B)
    assert np.array_equal(oracle.gemm_s8(M, N, K, A, Bb, layout_b=BLOCKED32), want)
    rows = np.array([36, 0, 5, 5], dtype=np.int64)
    assert np.array_equal(oracle.gemm_s8(M, N, K, A, Bb, layout_b=BLOCKED32, rows=rows, nthreads=3), want[rows])
    # identity: A . I = A; extremes: (-128) . (-128) summed K times
    eye = np.eye(K, dtype=np.int8)
    assert np.array_equal(oracle.gemm_s8(M, K, K, A, eye), A.astype(np.int64))
    lo = np.full((2, K), -128, dtype=np.int8)
    assert np.array_equal(oracle.gemm_s8(2, N, K, lo, np.full((K, N), -128, dtype=np.int8)),
                          np.full((2, N), 16384 * K, dtype=np.int64))
    # non-square roles: a transposed operand is caught
    assert not np.array_equal(oracle.gemm_s8(M, N, K, A, np.ascontiguousarray(B.T).reshape(K, N)), want)


def test_s8_planted_mistake_in_the_quad_order_is_caught():
    rng = np.random.default_rng(8)
    K, N = 32, 32
    A = rng.integers(-128, 128, (4, K), dtype=np.int8)
    B = rng.integers(-128, 128, (K, N), dtype=np.int8)
    good = oracle.to_blocked_s8(B)
    bad = good.reshape(-1, 4)[:, [1, 0, 2, 3]].reshape(-1)        # first two k of every quadruple swapped
    want = oracle.gemm_s8(4, N, K, A, B)
    assert np.array_equal(oracle.gemm_s8(4, N, K, A, good, layout_b=BLOCKED32), want)
    assert not np.array_equal(oracle.gemm_s8(4, N, K, A, np.ascontiguousarray(bad), layout_b=BLOCKED32), want)


def test_s8_generator_covers_the_range():
    v = nk_inputs.fill(11, nk_inputs.TENSOR_A, 1 << 16, dtype="s8")
    assert v.dtype == np.int8 and v.min() == -128 and v.max() == 127
    assert abs(float(v.astype(np.float64).mean())) < 1.5
    assert np.array_equal(v[100:200], nk_inputs.fill(11, nk_inputs.TENSOR_A, 100, dtype="s8", start=100))


def test_quantize_s8_ties_saturation_and_nan():
    x = np.array([0.5, 1.5, 2.5, -0.5, -1.5, -2.5, 0.49999997, 126.5, 127.5, 1e9, -128.5, -129.0, -1e9,
                  np.nan, 3.0, -0.0], dtype=np.float32)
    want = np.array([0, 2, 2, 0, -2, -2, 0, 126, 127, 127, -128, -128, -128, 0, 3, 0], dtype=np.int8)
    assert np.array_equal(oracle.quantize_s8(x, 1.0), want)
    # a power-of-two step is exact: x / 2^-4 = 16 x
    v = np.array([0.0625, 0.09375, -0.15625, 7.9375, 8.0], dtype=np.float32)       # 1, 1.5, -2.5, 127, 128 steps
    assert np.array_equal(oracle.quantize_s8(v, 16.0), np.array([1, 2, -2, 127, 127], dtype=np.int8))
    # against numpy's own float32 product and rint (round half to even), on random data
    rng = np.random.default_rng(9)
    r = (rng.standard_normal(4096) * 60).astype(np.float32)
    inv = np.float32(1.0 / 0.37)
    ref = np.clip(np.rint(r * inv), -128, 127).astype(np.int8)
    assert np.array_equal(oracle.quantize_s8(r, inv), ref)


def test_s8_scaled_layer_closed_forms():
    rng = np.random.default_rng(10)
    M, N, K = 8, 32, 64
    A = rng.integers(-128, 128, (M, K), dtype=np.int8)
    B = rng.integers(-128, 128, (K, N), dtype=np.int8)
    acc = A.astype(np.int64) @ B.astype(np.int64)
    y, s = oracle.gemm_s8_scaled(M, N, K, A, B, 0.5)
    assert np.array_equal(y, 0.5 * acc) and np.array_equal(s, np.abs(0.5 * acc))
    bias = -(0.25 * acc[0]).astype(np.float32)                # exact in FP32: |acc| < 2^21
    y, s = oracle.gemm_s8_scaled(M, N, K, A, B, 0.25, bias=bias, relu=True)
    assert np.all(y[0] == 0.0) and np.all(y >= 0.0)
    assert np.array_equal(s[0], 2 * np.abs(0.25 * acc[0]))


# ---------------------------------------------------------------- 8-bit floating point (E4M3, E5M2)
def test_fp8_decode_exhaustive_against_the_format_and_a_library():
    import torch
    bits = np.arange(256, dtype=np.uint8)
    sign = np.where(bits >> 7, -1.0, 1.0)
    # E4M3: bias 7, 3 fraction bits, no infinities, NaN only at exponent 15 / fraction 7
    e, m = ((bits >> 3) & 0xF).astype(np.int64), (bits & 7).astype(np.float64)
    want = np.where(e == 0, sign * m * 2.0 ** -9, sign * (1 + m / 8) * 2.0 ** (e - 7))
    got = oracle.fp8_to_f32(bits, oracle.E4M3).astype(np.float64)
    nan = (e == 15) & (m == 7)
    assert np.all(np.isnan(got[nan])) and np.array_equal(got[~nan], want[~nan])
    lib8 = torch.from_numpy(bits).view(torch.float8_e4m3fn).to(torch.float32).numpy().astype(np.float64)
    assert np.array_equal(got[~nan], lib8[~nan])
    assert got[0x38] == 1.0 and got[0x7E] == 448.0 and got[0x01] == 2.0 ** -9 and got[0xC0] == -2.0
    # E5M2: bias 15, 2 fraction bits, IEEE infinities and NaNs
    e, m = ((bits >> 2) & 0x1F).astype(np.int64), (bits & 3).astype(np.float64)
    want = np.where(e == 0, sign * m * 2.0 ** -16, sign * (1 + m / 4) * 2.0 ** (e - 15))
    got = oracle.fp8_to_f32(bits, oracle.E5M2).astype(np.float64)
    fin = e != 31
    assert np.array_equal(got[fin], want[fin])
    assert np.isposinf(got[0x7C]) and np.isneginf(got[0xFC]) and np.all(np.isnan(got[[0x7D, 0x7E, 0x7F, 0xFD]]))
    lib8 = torch.from_numpy(bits).view(torch.float8_e5m2).to(torch.float32).numpy().astype(np.float64)
    assert np.array_equal(got[fin], lib8[fin])
    assert got[0x3C] == 1.0 and got[0x7B] == 57344.0 and got[0x01] == 2.0 ** -16


@pytest.mark.parametrize("fmt", ["e4m3", "e5m2"])
def test_fp8_generator_rounds_to_nearest_even(fmt):
    import torch
    of, td, top = (oracle.E4M3, torch.float8_e4m3fn, 448.0) if fmt == "e4m3" else (oracle.E5M2, torch.float8_e5m2, 57344.0)
    rng = np.random.default_rng(12)
    v = np.concatenate([(rng.standard_normal(50000) * sc).astype(np.float32) for sc in (1.0, 0.02, 30.0, 1e-3)]
                       + [nk_inputs.fill(4, 0, 20000, "uniform", dtype="f32")])
    h = nk_inputs.f32_to_fp8_bits(v, fmt)
    # nearest: no other representable value is closer (checked through the decode of the neighbouring patterns)
    back = oracle.fp8_to_f32(h, of).astype(np.float64)
    mag = (h & 0x7F).astype(np.int64)
    up = oracle.fp8_to_f32(np.minimum(mag + 1, 0x7E if fmt == "e4m3" else 0x7B).astype(np.uint8), of).astype(np.float64)
    dn = oracle.fp8_to_f32(np.maximum(mag - 1, 0).astype(np.uint8), of).astype(np.float64)
    x = np.abs(np.clip(v.astype(np.float64), -top, top))
    assert np.all(np.abs(np.abs(back) - x) <= np.abs(up - x)) and np.all(np.abs(np.abs(back) - x) <= np.abs(dn - x))
    # ties go to the even pattern; the library's conversion agrees everywhere
    ref = torch.from_numpy(np.clip(v, -top, top)).to(td).view(torch.uint8).numpy()
    assert np.array_equal(h, ref)
    ties = np.array([1.0625, 1.1875, -1.1875], dtype=np.float32) if fmt == "e4m3" else np.array([1.125, 1.375, -1.375], dtype=np.float32)
    want = np.array([1.0, 1.25, -1.25]) if fmt == "e4m3" else np.array([1.0, 1.5, -1.5])
    assert np.array_equal(oracle.fp8_to_f32(nk_inputs.f32_to_fp8_bits(ties, fmt), of).astype(np.float64), want)


@pytest.mark.parametrize("fmt", ["e4m3", "e5m2"])
def test_fp8_gemm_equals_gemm_of_the_widened_operands(fmt):
    """8-bit floating-point operands, B row-major and blocked in groups of four, FP32 bias: the oracle on the
    8-bit storage equals, bit for bit, the oracle on the same values held as FP32 in row-major order."""
    M, N, K = 48, 64, 96
    of = oracle.E4M3 if fmt == "e4m3" else oracle.E5M2
    w = nk_inputs.Workload("t", M, N, K, fmt, "f32", layout="row", epilogue="bias_relu", seed=13)
    A, Bflat, bias = w.make()
    assert bias.dtype == np.float32
    Af, Bf = oracle.fp8_to_f32(A, of), oracle.fp8_to_f32(Bflat, of)
    Y0, S0 = oracle.gemm(M, N, K, Af, Bf, bias, in_dtype=F32, epilogue=EPI_BIAS_RELU)
    Y1, S1 = oracle.gemm_workload(w, A, Bflat, bias)
    assert np.array_equal(Y0, Y1) and np.array_equal(S0, S1)
    # blocked B: the bytes scattered by the INT8 rule (groups of four inside 32 x 32 blocks)
    Bblk = oracle.to_blocked_s8(Bflat.reshape(K, N).view(np.int8)).view(np.uint8)
    wb = nk_inputs.Workload("t", M, N, K, fmt, "f32", layout="b_blocked32", epilogue="bias_relu", seed=13)
    Y2, S2 = oracle.gemm_workload(wb, A, Bblk, bias)
    assert np.array_equal(Y0, Y2) and np.array_equal(S0, S2)
    assert np.abs(Y0 - np.maximum(Af.astype(np.float64).reshape(M, K) @ Bf.astype(np.float64).reshape(K, N) + bias, 0)).max() < 1e-9


# ---------------------------------------------------------------- B kept as its transpose
def test_transposed_b_is_the_same_matrix():
    """layout_b = TRANSPOSED only changes where element (k, j) of B is stored: the oracle on Bt[N][K] equals,
    bit for bit, the oracle on B[K][N]; and giving it B untransposed is caught."""
    rng = np.random.default_rng(14)
    M, N, K = 24, 40, 56
    A = rng.standard_normal((M, K)).astype(np.float32)
    B = rng.standard_normal((K, N)).astype(np.float32)
    Y0, S0 = oracle.gemm(M, N, K, A, B)
    Y1, S1 = oracle.gemm(M, N, K, A, np.ascontiguousarray(B.T), layout_b=oracle.TRANSPOSED)
    assert np.array_equal(Y0, Y1) and np.array_equal(S0, S1)
    Y2, _ = oracle.gemm(M, N, K, A, B, layout_b=oracle.TRANSPOSED)
    assert not np.array_equal(Y0, Y2)
    A8 = rng.integers(-128, 128, (M, K), dtype=np.int8)
    B8 = rng.integers(-128, 128, (K, N), dtype=np.int8)
    want = A8.astype(np.int64) @ B8.astype(np.int64)
    assert np.array_equal(oracle.gemm_s8(M, N, K, A8, np.ascontiguousarray(B8.T), layout_b=oracle.TRANSPOSED), want)
