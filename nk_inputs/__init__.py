"""Seeded synthetic operands for the dense-GEMM path.

This module only draws numbers and names workloads.  It holds no GEMM
arithmetic, no layout packing and no epilogue: both the CUDA library's tests
and the CPU oracle's tests take their inputs from here so that they see the
same bits, and neither implementation depends on the other.

Generator (counter based, stateless): the value at flat storage index ``idx``
of tensor ``tensor_id`` under ``seed`` depends only on those three integers,

    h = mix64(mix64(seed * GOLDEN + tensor_id) + idx)

with ``mix64`` the SplitMix64 output function (Steele, Lea & Flood 2014).
Uniform values take the top 24 bits of ``h``: ``u = t * 2**-23 - 1`` lies in
[-1, 1) and is exact in FP32.  Normal values use Box-Muller in float64 on two
independent 53/24-bit draws.  BF16 tensors are the FP32 draw rounded to
nearest-even and returned as raw ``uint16`` bit patterns.

Tensors are generated in *storage order*: entries are i.i.d., so a blocked or
VNNI-packed operand is simply a buffer of the right length filled by index;
no packing routine is needed to make inputs.
"""
from __future__ import annotations

import dataclasses
import numpy as np

GOLDEN = np.uint64(0x9E3779B97F4A7C15)
TENSOR_A, TENSOR_B, TENSOR_BIAS, TENSOR_ROWS, TENSOR_VEC = 0, 1, 2, 8, 9

_CHUNK = 1 << 22


def mix64(z: np.ndarray) -> np.ndarray:
    """SplitMix64 finaliser on a uint64 array (wrap-around arithmetic)."""
    z = z.astype(np.uint64, copy=True)
    with np.errstate(over="ignore"):
        z ^= z >> np.uint64(30)
        z *= np.uint64(0xBF58476D1CE4E5B9)
        z ^= z >> np.uint64(27)
        z *= np.uint64(0x94D049BB133111EB)
        z ^= z >> np.uint64(31)
    return z


def _stream_key(seed: int, tensor_id: int) -> np.uint64:
    with np.errstate(over="ignore"):
        k = np.uint64(seed) * GOLDEN + np.uint64(tensor_id)
    return mix64(np.array([k], dtype=np.uint64))[0]


def raw_bits(seed: int, tensor_id: int, start: int, count: int) -> np.ndarray:
    """64 random bits for storage indices start .. start+count-1."""
    key = _stream_key(seed, tensor_id)
    idx = np.arange(start, start + count, dtype=np.uint64)
    with np.errstate(over="ignore"):
        return mix64(idx + key)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round finite FP32 values to BF16 (nearest, ties to even); returns uint16."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = u + np.uint32(0x7FFF) + lsb
    return (r >> np.uint32(16)).astype(np.uint16)


def f32_to_f16_bits(x: np.ndarray) -> np.ndarray:
    """Round finite FP32 values to IEEE binary16 (nearest, ties to even); returns uint16."""
    return np.ascontiguousarray(x, dtype=np.float32).astype(np.float16).view(np.uint16)


def _uniform_f32(seed, tensor_id, start, count):
    t = (raw_bits(seed, tensor_id, start, count) >> np.uint64(40)).astype(np.float64)
    return (t * 2.0 ** -23 - 1.0).astype(np.float32)


def _normal_f32(seed, tensor_id, start, count, sigma):
    h = raw_bits(seed, tensor_id, start, count)
    # two draws per element: 32 high bits -> radius, 32 low bits -> angle
    u1 = ((h >> np.uint64(32)).astype(np.float64) + 1.0) * 2.0 ** -32      # (0, 1]
    u2 = (h & np.uint64(0xFFFFFFFF)).astype(np.float64) * 2.0 ** -32       # [0, 1)
    z = np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)
    return (z * sigma).astype(np.float32)


def f32_to_fp8_bits(v: np.ndarray, fmt: str) -> np.ndarray:
    """FP32 -> 8-bit floating point ("e4m3": 4 exponent bits, bias 7, 3 fraction bits, largest finite
    value 448; "e5m2": 5 exponent bits, bias 15, 2 fraction bits, largest finite value 57344), round to
    nearest, ties to even, gradual underflow, finite inputs; magnitudes beyond the largest finite value
    saturate to it."""
    man, bias, emin, top = (3, 7, -6, 448.0) if fmt == "e4m3" else (2, 15, -14, 57344.0)
    x = np.minimum(np.abs(v.astype(np.float64)), top)
    _, E = np.frexp(x)                              # x = m * 2^E, m in [0.5, 1)
    e = np.maximum(E - 1, emin)                     # exponent of the binade (subnormals share emin)
    q = np.rint(x / np.exp2((e - man).astype(np.float64))).astype(np.int64)   # significand in units of 2^(e - man): ties to even
    # q may reach 2^(man+1) (carry into the next binade): the bit arithmetic below absorbs it
    bits = ((e - emin) << man) + q                  # subnormals: exponent field 0, q < 2^man; normals: field (e - emin + 1), q - 2^man
    bits = np.where(x == 0, 0, bits)
    sign = (np.signbit(v)).astype(np.int64) << 7
    return (bits | sign).astype(np.uint8)


def fill(seed: int, tensor_id: int, count: int, dist: str = "uniform",
         sigma: float = 1.0, dtype: str = "f32", start: int = 0) -> np.ndarray:
    """1-D storage-order buffer of ``count`` entries (storage indices start .. start+count-1).

    dist: "uniform" (U[-1,1) on the 2**-23 grid), "normal" (N(0, sigma**2)),
          "int" (integers in [-4, 4], exact in every precision used here).
    dtype: "f32" -> float32 array; "bf16" / "f16" -> uint16 bit patterns; "s8" -> int8, uniform over
           all 256 values; "e4m3" / "e5m2" -> uint8 bit patterns of the 8-bit floating-point formats.
    """
    if dtype == "s8":
        # INT8 operands: the full range [-128, 127], uniformly, whatever `dist` says
        out = np.empty(count, dtype=np.int8)
        for s in range(0, count, _CHUNK):
            n = min(_CHUNK, count - s)
            out[s:s + n] = ((raw_bits(seed, tensor_id, start + s, n) >> np.uint64(40)) & np.uint64(0xFF)
                            ).astype(np.uint8).view(np.int8)
        return out
    out = np.empty(count, dtype=np.float32 if dtype == "f32" else np.uint8 if dtype in ("e4m3", "e5m2") else np.uint16)
    for s in range(0, count, _CHUNK):
        n = min(_CHUNK, count - s)
        if dist == "uniform":
            v = _uniform_f32(seed, tensor_id, start + s, n)
        elif dist == "normal":
            v = _normal_f32(seed, tensor_id, start + s, n, sigma)
        elif dist == "int":
            v = ((raw_bits(seed, tensor_id, start + s, n) >> np.uint64(40)) % np.uint64(9)
                 ).astype(np.float32) - 4.0
        else:
            raise ValueError(dist)
        out[s:s + n] = (v if dtype == "f32" else f32_to_f16_bits(v) if dtype == "f16"
                        else f32_to_fp8_bits(v, dtype) if dtype in ("e4m3", "e5m2") else f32_to_bf16_bits(v))
    return out


def stratified_rows(seed: int, M: int, n: int = 64) -> np.ndarray:
    """``n`` row indices, one per equal band of [0, M): band t contributes
    t*band + (hash mod band).  For M = 8192, n = 64 every 128-row tile is hit."""
    n = min(n, M)
    band = M // n
    h = raw_bits(seed, TENSOR_ROWS, 0, n)
    rows = np.arange(n, dtype=np.int64) * band + (h % np.uint64(band)).astype(np.int64)
    return rows


def sample_cols(seed: int, N: int, n: int) -> np.ndarray:
    """``n`` distinct sorted column indices (all of them when n >= N)."""
    if n >= N:
        return np.arange(N, dtype=np.int64)
    band = N // n
    h = raw_bits(seed, TENSOR_VEC, 0, n)
    return np.arange(n, dtype=np.int64) * band + (h % np.uint64(band)).astype(np.int64)


@dataclasses.dataclass(frozen=True)
class Workload:
    """One GEMM problem: shapes, element types, operand layouts, epilogue,
    and the distributions its operands are drawn from."""
    name: str
    M: int
    N: int
    K: int
    in_dtype: str = "bf16"          # "f32" | "bf16" | "f16" | "s8"
    out_dtype: str = "f32"          # "f32" | "bf16" | "f16" (a 16-bit output has the input's type) | "s32" (INT8 operands)
    layout: str = "row"             # "row" | "blocked32" (A and B both) | "b_blocked32" (A row-major, B blocked)
                                    # | "b_transposed" (A row-major, B kept as Bt[N][K])
    epilogue: str = "none"          # "none" | "bias_relu"
    dist_a: tuple = ("uniform", 1.0)
    dist_b: tuple = ("uniform", 1.0)
    dist_bias: tuple = ("normal", 0.02)
    seed: int = 17

    @property
    def flops(self) -> float:
        return 2.0 * self.M * self.N * self.K

    @property
    def algorithmic_bytes(self) -> int:
        e_in = 4 if self.in_dtype == "f32" else 1 if self.in_dtype in ("s8", "e4m3", "e5m2") else 2
        e_out = 4 if self.out_dtype in ("f32", "s32") else 2
        b = e_in * (self.M * self.K + self.K * self.N) + e_out * self.M * self.N
        if self.epilogue != "none":
            b += (4 if self.in_dtype in ("e4m3", "e5m2") else e_in) * self.N
        return b

    def make(self):
        """Returns (A, B, bias) as 1-D numpy storage buffers (bias None when
        there is no epilogue).  Blocked layouts have the same element count as
        row-major; only the meaning of the storage index differs."""
        A = fill(self.seed, TENSOR_A, self.M * self.K, self.dist_a[0], self.dist_a[1], self.in_dtype)
        B = fill(self.seed, TENSOR_B, self.K * self.N, self.dist_b[0], self.dist_b[1], self.in_dtype)
        bias = None
        if self.epilogue != "none":
            bias = fill(self.seed, TENSOR_BIAS, self.N, self.dist_bias[0], self.dist_bias[1], self.bias_dtype)
        return A, B, bias

    @property
    def bias_dtype(self) -> str:
        """The bias has the operands' type, except with 8-bit floating-point operands (FP32 bias)."""
        return "f32" if self.in_dtype in ("e4m3", "e5m2") else self.in_dtype


def config(i: int) -> Workload:
    """The four fixed benchmark configurations (1-based, seeds 1000*i + 17)."""
    s = 1000 * i + 17
    if i == 1:
        return Workload("c1_f32_256", 256, 256, 256, "f32", "f32", seed=s)
    if i == 2:
        return Workload("c2_bf16_blocked_1024", 1024, 1024, 1024, "bf16", "f32", layout="blocked32", seed=s)
    if i == 3:
        return Workload("c3_bf16_mlp_256x4096x4096", 256, 4096, 4096, "bf16", "bf16",
                        epilogue="bias_relu", dist_a=("normal", 1.0), dist_b=("normal", 0.02), seed=s)
    if i == 4:
        return Workload("c4_bf16_8192", 8192, 8192, 8192, "bf16", "f32", seed=s)
    raise ValueError(i)


def sweep() -> list:
    """Configuration 5: M in {16,128,1024,4096} x N=K in {1024,4096,16384}, both dtypes."""
    out = []
    for dt in ("f32", "bf16"):
        for nk in (1024, 4096, 16384):
            for m in (16, 128, 1024, 4096):
                out.append(Workload(f"c5_{dt}_{m}x{nk}x{nk}", m, nk, nk, dt, "f32",
                                    seed=5017 + nk))      # B is shared by the four M values
    return out


def paper_mlp() -> list:
    """The paper's own MLP grid (Section 6): batch 512, layer size 1024/2048/4096,
    FP32 / BF16 VNNI-blocked / BF16 flat, bias + ReLU."""
    out = []
    for n in (1024, 2048, 4096):
        out.append(Workload(f"mlp_f32_{n}", 512, n, n, "f32", "f32", epilogue="bias_relu",
                            dist_a=("normal", 1.0), dist_b=("normal", 0.02), seed=6000 + n))
        out.append(Workload(f"mlp_bf16_vnni_{n}", 512, n, n, "bf16", "bf16", layout="blocked32",
                            epilogue="bias_relu", dist_a=("normal", 1.0), dist_b=("normal", 0.02),
                            seed=6001 + n))
        out.append(Workload(f"mlp_bf16_flat_{n}", 512, n, n, "bf16", "bf16", epilogue="bias_relu",
                            dist_a=("normal", 1.0), dist_b=("normal", 0.02), seed=6002 + n))
    return out


def s8_set() -> list:
    """INT8 operands (the Int8 dot product Section 5 names as the next packed type), B packed in
    groups of four inside 32 x 32 blocks, INT32 result: the large square GEMM, a mid-size one and
    the paper's 4096-wide MLP layer shape."""
    return [
        Workload("x_s8_8192", 8192, 8192, 8192, "s8", "s32", layout="b_blocked32", seed=8017),
        Workload("x_s8_4096", 4096, 4096, 4096, "s8", "s32", layout="b_blocked32", seed=8018),
        Workload("x_s8_512x4096x4096", 512, 4096, 4096, "s8", "s32", layout="b_blocked32", seed=8019),
    ]


def fp8_set() -> list:
    """8-bit floating-point operands (E4M3 / E5M2; the 8-bit floating-point counterpart, on B200, of the
    packed types Section 5 lists), B packed in groups of four inside 32 x 32 blocks, FP32 accumulation
    and output: the large square GEMM, a mid-size E5M2 one and the 4096-wide MLP layer with FP32 bias."""
    return [
        Workload("x_e4m3_8192", 8192, 8192, 8192, "e4m3", "f32", layout="b_blocked32", seed=9017),
        Workload("x_e5m2_4096", 4096, 4096, 4096, "e5m2", "f32", layout="b_blocked32", seed=9018),
        Workload("x_e4m3_mlp_512x4096x4096", 512, 4096, 4096, "e4m3", "f32", layout="b_blocked32", epilogue="bias_relu",
                 dist_a=("normal", 1.0), dist_b=("normal", 0.02), seed=9019),
    ]


def bt_set() -> list:
    """B kept as its transpose Bt[N][K] (the form a linear layer's weight usually has): the large square GEMM
    in BF16, INT8 and E4M3."""
    return [
        Workload("xt_bf16_8192", 8192, 8192, 8192, "bf16", "f32", layout="b_transposed", seed=9517),
        Workload("xt_s8_8192", 8192, 8192, 8192, "s8", "s32", layout="b_transposed", seed=9518),
        Workload("xt_e4m3_8192", 8192, 8192, 8192, "e4m3", "f32", layout="b_transposed", seed=9519),
        Workload("xt_s8_4096", 4096, 4096, 4096, "s8", "s32", layout="b_transposed", seed=9520),
    ]


def f16_set() -> list:
    """FP16 (IEEE binary16) counterparts of the headline shapes: the large square GEMM, the MLP
    layer of configuration 3, and the paper's 4096-wide MLP layer."""
    return [
        Workload("x_f16_8192", 8192, 8192, 8192, "f16", "f32", seed=7017),
        Workload("x_f16_mlp_256x4096x4096", 256, 4096, 4096, "f16", "f16", epilogue="bias_relu",
                 dist_a=("normal", 1.0), dist_b=("normal", 0.02), seed=7018),
        Workload("x_f16_mlp_512x4096x4096", 512, 4096, 4096, "f16", "f16", epilogue="bias_relu",
                 dist_a=("normal", 1.0), dist_b=("normal", 0.02), seed=7019),
    ]
