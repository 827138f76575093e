"""Python face of the CPU oracle (``nk_oracle.c``).

TEST INFRASTRUCTURE ONLY.  Tests, the smoke check and the benchmark's CPU
baseline leg may import this package; the product package never does, and this
package never imports the product.  It compiles ``nk_oracle.c`` with gcc on
first use and calls it through ctypes; the arithmetic lives in the C file.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "nk_oracle.c")
_LIB = os.path.join(_HERE, "libnk_oracle.so")

F32, BF16, F16 = 0, 1, 2
E4M3, E5M2 = 5, 6
ROW, BLOCKED32, TRANSPOSED = 0, 1, 2
EPI_NONE, EPI_BIAS_RELU = 0, 1
ACC_F64, ACC_F32_SEQ = 0, 1


class Desc(ctypes.Structure):
    _fields_ = [("M", ctypes.c_int64), ("N", ctypes.c_int64), ("K", ctypes.c_int64),
                ("in_dtype", ctypes.c_int32), ("layout_a", ctypes.c_int32),
                ("layout_b", ctypes.c_int32), ("epilogue", ctypes.c_int32),
                ("acc_mode", ctypes.c_int32)]


def build(force: bool = False) -> str:
    """Compile the oracle's C file (plain gcc, -O2, no fast-math)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-pthread",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        L.nko_bf16_to_f32.restype = ctypes.c_float
        L.nko_bf16_to_f32.argtypes = [ctypes.c_uint16]
        L.nko_f16_to_f32.restype = ctypes.c_float
        L.nko_f16_to_f32.argtypes = [ctypes.c_uint16]
        for f in (L.nko_e4m3_to_f32, L.nko_e5m2_to_f32):
            f.restype = ctypes.c_float
            f.argtypes = [ctypes.c_uint8]
        L.nko_f32_to_bf16_rne.restype = ctypes.c_uint16
        L.nko_f32_to_bf16_rne.argtypes = [ctypes.c_float]
        for f in (L.nko_pack_vnni2, L.nko_unpack_vnni2):
            f.restype = None
            f.argtypes = [ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64, ctypes.c_void_p]
        for f in (L.nko_a_index, L.nko_b_index):
            f.restype = ctypes.c_int64
            f.argtypes = [ctypes.POINTER(Desc), ctypes.c_int64, ctypes.c_int64]
        L.nko_gemm.restype = ctypes.c_int
        L.nko_gemm.argtypes = [ctypes.POINTER(Desc), ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                               ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p, ctypes.c_int64,
                               ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int]
        L.nko_brgemm.restype = ctypes.c_int
        L.nko_brgemm.argtypes = [ctypes.c_int64] * 6 + [ctypes.c_int32, ctypes.c_int32, ctypes.c_double,
                                 ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                 ctypes.c_void_p, ctypes.c_void_p]
        L.nko_brgemm_layout.restype = ctypes.c_int
        L.nko_brgemm_layout.argtypes = [ctypes.c_int64] * 6 + [ctypes.c_int32] * 4 + [ctypes.c_double,
                                        ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                        ctypes.c_void_p, ctypes.c_void_p]
        for f in (L.nko_pack_vnni4, L.nko_unpack_vnni4):
            f.restype = None
            f.argtypes = [ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64, ctypes.c_void_p]
        L.nko_b_index_s8.restype = ctypes.c_int64
        L.nko_b_index_s8.argtypes = [ctypes.c_int64, ctypes.c_int64, ctypes.c_int32, ctypes.c_int64, ctypes.c_int64]
        L.nko_quantize_s8.restype = None
        L.nko_quantize_s8.argtypes = [ctypes.c_void_p, ctypes.c_int64, ctypes.c_float, ctypes.c_void_p]
        L.nko_gemm_s8.restype = ctypes.c_int
        L.nko_gemm_s8.argtypes = [ctypes.c_int64, ctypes.c_int64, ctypes.c_int64, ctypes.c_int32, ctypes.c_void_p,
                                  ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p, ctypes.c_int]
        _lib = L
    return _lib


def pack_vnni4(flat: np.ndarray) -> np.ndarray:
    """[K][N] int8 -> [K/4][N][4]: Figure 1's rule with groups of four (Section 2)."""
    flat = np.ascontiguousarray(flat, dtype=np.int8)
    K, N = flat.shape
    assert K % 4 == 0
    out = np.empty((K // 4, N, 4), dtype=np.int8)
    lib().nko_pack_vnni4(flat.ctypes.data, K, N, out.ctypes.data)
    return out


def unpack_vnni4(packed: np.ndarray) -> np.ndarray:
    packed = np.ascontiguousarray(packed, dtype=np.int8)
    K4, N, four = packed.shape
    assert four == 4
    out = np.empty((K4 * 4, N), dtype=np.int8)
    lib().nko_unpack_vnni4(packed.ctypes.data, K4 * 4, N, out.ctypes.data)
    return out


def to_blocked_s8(flat_b: np.ndarray) -> np.ndarray:
    """Scatter a row-major int8 B[K][N] into B_blk4[N/32][K/32][8][32][4] with the oracle's own
    index function (Python loop; test sizes only)."""
    K, N = flat_b.shape
    L = lib()
    B = np.empty(K * N, dtype=np.int8)
    for k in range(K):
        for j in range(N):
            B[L.nko_b_index_s8(K, N, BLOCKED32, k, j)] = flat_b[k, j]
    return B


def gemm_s8(M, N, K, A, B, *, layout_b=ROW, rows=None, nthreads=None) -> np.ndarray:
    """Exact integer product of int8 operands: int64 [rows][N] (all M rows by default)."""
    A = np.ascontiguousarray(A, dtype=np.int8).ravel()
    B = np.ascontiguousarray(B, dtype=np.int8).ravel()
    assert A.size == M * K and B.size == K * N
    r = None if rows is None else np.ascontiguousarray(rows, dtype=np.int64)
    nr = M if r is None else r.size
    Y = np.empty((nr, N), dtype=np.int64)
    nt = nthreads or min(os.cpu_count() or 1, 32)
    rc = lib().nko_gemm_s8(M, N, K, layout_b, A.ctypes.data, B.ctypes.data, None if r is None else r.ctypes.data,
                           nr, Y.ctypes.data, nt)
    if rc != 0:
        raise ValueError("nko_gemm_s8: bad arguments")
    return Y


def bf16_to_f32(bits: np.ndarray) -> np.ndarray:
    """Decode uint16 BF16 patterns element by element through the C routine."""
    L = lib()
    flat = np.ascontiguousarray(bits, dtype=np.uint16).ravel()
    out = np.fromiter((L.nko_bf16_to_f32(int(h)) for h in flat), dtype=np.float32, count=flat.size)
    return out.reshape(np.shape(bits))


def f16_to_f32(bits: np.ndarray) -> np.ndarray:
    """Decode uint16 IEEE binary16 patterns element by element through the C routine."""
    L = lib()
    flat = np.ascontiguousarray(bits, dtype=np.uint16).ravel()
    out = np.fromiter((L.nko_f16_to_f32(int(h)) for h in flat), dtype=np.float32, count=flat.size)
    return out.reshape(np.shape(bits))


def f32_to_bf16_rne(x: np.ndarray) -> np.ndarray:
    L = lib()
    flat = np.ascontiguousarray(x, dtype=np.float32).ravel()
    out = np.fromiter((L.nko_f32_to_bf16_rne(float(v)) for v in flat), dtype=np.uint16, count=flat.size)
    return out.reshape(np.shape(x))


def pack_vnni2(flat: np.ndarray) -> np.ndarray:
    """[K][N] uint16 -> [K/2][N][2] (Figure 1)."""
    flat = np.ascontiguousarray(flat, dtype=np.uint16)
    K, N = flat.shape
    assert K % 2 == 0
    out = np.empty((K // 2, N, 2), dtype=np.uint16)
    lib().nko_pack_vnni2(flat.ctypes.data, K, N, out.ctypes.data)
    return out


def unpack_vnni2(packed: np.ndarray) -> np.ndarray:
    packed = np.ascontiguousarray(packed, dtype=np.uint16)
    K2, N, two = packed.shape
    assert two == 2
    out = np.empty((K2 * 2, N), dtype=np.uint16)
    lib().nko_unpack_vnni2(packed.ctypes.data, K2 * 2, N, out.ctypes.data)
    return out


def _np_dtype(in_dtype):
    return np.float32 if in_dtype == F32 else np.uint8 if in_dtype in (E4M3, E5M2) else np.uint16


def fp8_to_f32(bits: np.ndarray, fmt: int) -> np.ndarray:
    """Decode uint8 E4M3 / E5M2 patterns element by element through the C routines."""
    L = lib()
    f = L.nko_e4m3_to_f32 if fmt == E4M3 else L.nko_e5m2_to_f32
    flat = np.ascontiguousarray(bits, dtype=np.uint8).ravel()
    out = np.fromiter((f(int(h)) for h in flat), dtype=np.float32, count=flat.size)
    return out.reshape(np.shape(bits))


def to_blocked(flat_a: np.ndarray, flat_b: np.ndarray, in_dtype: int):
    """Scatter row-major A[M][K], B[K][N] into the blocked storage order using the
    oracle's own index functions (slow Python loop over rows; test sizes only)."""
    M, K = flat_a.shape
    K2, N = flat_b.shape
    assert K == K2
    d = Desc(M, N, K, in_dtype, BLOCKED32, BLOCKED32, EPI_NONE, ACC_F64)
    L = lib()
    A = np.empty(M * K, dtype=flat_a.dtype)
    B = np.empty(K * N, dtype=flat_b.dtype)
    for i in range(M):
        for k in range(K):
            A[L.nko_a_index(ctypes.byref(d), i, k)] = flat_a[i, k]
    for k in range(K):
        for j in range(N):
            B[L.nko_b_index(ctypes.byref(d), k, j)] = flat_b[k, j]
    return A, B


def gemm(M, N, K, A, B, bias=None, *, in_dtype=F32, layout_a=ROW, layout_b=ROW,
         epilogue=EPI_NONE, rows=None, cols=None, acc_mode=ACC_F64, nthreads=None,
         want_scale=True):
    """Run the oracle.  A, B, bias are 1-D (or any-shape, C-contiguous) storage
    buffers: float32, or uint16 BF16 bit patterns.  Returns (Y, S) as float64
    arrays of shape [len(rows) or M][len(cols) or N]; S is None when
    ``want_scale`` is False."""
    dt = _np_dtype(in_dtype)
    A = np.ascontiguousarray(A, dtype=dt)
    B = np.ascontiguousarray(B, dtype=dt)
    assert A.size == M * K and B.size == K * N, "operand size mismatch"
    bp = None
    if bias is not None:
        bias = np.ascontiguousarray(bias, dtype=np.float32 if in_dtype in (E4M3, E5M2) else dt)
        assert bias.size == N
        bp = bias.ctypes.data
    rp, nrows = None, M
    if rows is not None:
        rows = np.ascontiguousarray(rows, dtype=np.int64)
        assert rows.min() >= 0 and rows.max() < M
        rp, nrows = rows.ctypes.data, rows.size
    cp, ncols = None, N
    if cols is not None:
        cols = np.ascontiguousarray(cols, dtype=np.int64)
        assert cols.min() >= 0 and cols.max() < N
        cp, ncols = cols.ctypes.data, cols.size
    Y = np.empty((nrows, ncols), dtype=np.float64)
    S = np.empty((nrows, ncols), dtype=np.float64) if want_scale else None
    d = Desc(M, N, K, in_dtype, layout_a, layout_b, epilogue, acc_mode)
    if nthreads is None:
        nthreads = os.cpu_count() or 1
    rc = lib().nko_gemm(ctypes.byref(d), A.ctypes.data, B.ctypes.data, bp, rp, nrows, cp, ncols,
                        Y.ctypes.data, S.ctypes.data if S is not None else None, int(nthreads))
    if rc != 0:
        raise ValueError("oracle rejected the arguments")
    return Y, S


def gemm_workload(w, A, B, bias, rows=None, cols=None, **kw):
    """Oracle on an ``nk_inputs.Workload``-shaped object (duck-typed: M, N, K,
    in_dtype, layout, epilogue attributes)."""
    lay_a = BLOCKED32 if w.layout == "blocked32" else ROW
    lay_b = BLOCKED32 if w.layout in ("blocked32", "b_blocked32") else TRANSPOSED if w.layout == "b_transposed" else ROW
    return gemm(w.M, w.N, w.K, A, B, bias,
                in_dtype={"f32": F32, "bf16": BF16, "f16": F16, "e4m3": E4M3, "e5m2": E5M2}[w.in_dtype],
                layout_a=lay_a, layout_b=lay_b,
                epilogue=EPI_BIAS_RELU if w.epilogue == "bias_relu" else EPI_NONE,
                rows=rows, cols=cols, **kw)


def brgemm(M, N, K, batch, A, B, bias=None, C0=None, *, in_dtype=F32, epilogue=EPI_NONE, beta=0.0,
           stride_a=None, stride_b=None, layout_a=ROW, layout_b=ROW):
    """Batch-reduce GEMM (Algorithm 1's output line): beta*C0 + sum_b A_b.B_b.
    A and B are storage buffers holding all batch items (item b of A starts at b*stride_a
    elements; default M*K and K*N), every item row-major or 32x32-blocked / VNNI-packed
    (Listing 1's items).  C0: float64 [M][N] (the stored C widened) when beta = 1.
    Returns (Y, S) float64 [M][N]."""
    dt = _np_dtype(in_dtype)
    A = np.ascontiguousarray(A, dtype=dt)
    B = np.ascontiguousarray(B, dtype=dt)
    stride_a = M * K if stride_a is None else stride_a
    stride_b = K * N if stride_b is None else stride_b
    assert A.size >= (batch - 1) * stride_a + M * K and B.size >= (batch - 1) * stride_b + K * N
    bp = None
    if bias is not None:
        bias = np.ascontiguousarray(bias, dtype=dt)
        bp = bias.ctypes.data
    cp = None
    if C0 is not None:
        C0 = np.ascontiguousarray(C0, dtype=np.float64)
        assert C0.size == M * N
        cp = C0.ctypes.data
    Y = np.empty((M, N), dtype=np.float64)
    S = np.empty((M, N), dtype=np.float64)
    if layout_a == ROW and layout_b == ROW:
        rc = lib().nko_brgemm(M, N, K, batch, stride_a, stride_b, in_dtype, epilogue, float(beta),
                              A.ctypes.data, B.ctypes.data, bp, cp, Y.ctypes.data, S.ctypes.data)
    else:
        rc = lib().nko_brgemm_layout(M, N, K, batch, stride_a, stride_b, in_dtype, layout_a, layout_b, epilogue,
                                     float(beta), A.ctypes.data, B.ctypes.data, bp, cp, Y.ctypes.data, S.ctypes.data)
    if rc != 0:
        raise ValueError("oracle rejected the arguments")
    return Y, S


def quantize_s8(x: np.ndarray, inv_scale: float) -> np.ndarray:
    """FP32 -> INT8: saturate(round-half-even(fl32(x * inv_scale))); NaN -> 0."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    q = np.empty(x.shape, dtype=np.int8)
    lib().nko_quantize_s8(x.ctypes.data, x.size, float(np.float32(inv_scale)), q.ctypes.data)
    return q


def gemm_s8_scaled(M, N, K, A, B, scale, bias=None, *, layout_b=ROW, rows=None, relu=False):
    """The quantised layer on top of the exact integer product: y = scale * (A.B) (+ bias, then
    max(., 0)), in float64, with S = |scale * (A.B)| (+ |bias|) as the scale of the error bound."""
    acc = gemm_s8(M, N, K, A, B, layout_b=layout_b, rows=rows).astype(np.float64)
    y = float(np.float32(scale)) * acc
    s = np.abs(y)
    if bias is not None:
        b = np.asarray(bias, dtype=np.float32).astype(np.float64)
        y = y + b[None, :]
        s = s + np.abs(b)[None, :]
    if relu:
        y = np.maximum(y, 0.0)
    return y, s
