"""ctypes binding of include/nk_gemm.h.  Same names, argument marshalling only.

The binding loads the in-tree ``libnk_gemm.so`` and fails loudly when it is
missing or cannot be loaded: there is no Python or CPU fallback.
"""
from __future__ import annotations

import ctypes
import os

from . import _build

F32, BF16, F16, S8, S32, E4M3, E5M2 = 0, 1, 2, 3, 4, 5, 6
ROW_MAJOR, BLOCKED32, TRANSPOSED = 0, 1, 2
EPI_NONE, EPI_BIAS_RELU = 0, 1
FLAG_KERNEL_NAIVE, FLAG_KERNEL_SIMT, FLAG_KERNEL_UMMA = 0x1, 0x2, 0x3
FLAG_REPACK_B = 0x10
FLAG_SINGLE_CTA, FLAG_CTA_PAIR = 0x20, 0x40
FLAG_SCALAR_FMA = 0x80
FLAG_SEPARATE_REDUCE = 0x100000
FLAG_LSU_STORE = 0x200000
FLAG_NO_TAIL_SPLIT = 0x400000
FLAG_F32_TENSOR = 0x800000

EXPORTS = ["nk_gemm_create", "nk_gemm_workspace_bytes", "nk_gemm_run", "nk_gemm_run_host",
           "nk_gemm_check", "nk_gemm_destroy", "nk_status_str", "nk_gemm_kernel_name",
           "nk_gemm_launches_per_run", "nk_gemm_last_cuda_error", "nk_gemm_run_static",
           "nk_gemm_selftest_timeout", "nk_quantize_s8"]

STATIC_SCRATCH_BYTES = 16 << 20


def flag_splitk(n: int) -> int:
    return (n & 0xFF) << 8


def flag_tail_split(n: int) -> int:
    """Force n K splits (2..8) for the tiles of the last, partial wave (pair kernel)."""
    return (n & 0xF) << 24


def flag_raster(group_code: int, serpentine: bool = True) -> int:
    """Tile raster of the tensor-core kernels: group_code 0..6 = 8, 4, 6, 12, 16, 24, 2 M tiles per group;
    7 = 8 with K walked upwards on every tile (no K serpentine)."""
    return ((group_code & 7) << 28) | (0 if serpentine else (1 << 31))


def flag_tile_n(code: int) -> int:
    """1=32, 2=64, 3=128, 4=256."""
    return (code & 0xF) << 16


class NkError(RuntimeError):
    def __init__(self, status: int, msg: str):
        super().__init__(f"nk_gemm status {status}: {msg}")
        self.status = status


class Desc(ctypes.Structure):
    _fields_ = [("M", ctypes.c_int64), ("N", ctypes.c_int64), ("K", ctypes.c_int64),
                ("in_dtype", ctypes.c_int32), ("out_dtype", ctypes.c_int32),
                ("layout_a", ctypes.c_int32), ("layout_b", ctypes.c_int32),
                ("epilogue", ctypes.c_int32), ("device", ctypes.c_int32),
                ("flags", ctypes.c_uint32), ("beta", ctypes.c_int32), ("batch", ctypes.c_int64),
                ("stride_a", ctypes.c_int64), ("stride_b", ctypes.c_int64), ("stride_c", ctypes.c_int64),
                ("batch_independent", ctypes.c_int32), ("layout_c", ctypes.c_int32), ("scale", ctypes.c_float)]


_lib = None


def lib_path() -> str:
    return _build.LIB


def lib():
    """Load libnk_gemm.so, building it first when it is missing or was built from other
    sources than the ones in the tree now."""
    global _lib
    if _lib is None:
        path = _build.build(force=bool(os.environ.get("NK_GEMM_REBUILD")))
        L = ctypes.CDLL(path)          # raises OSError when unusable: no fallback
        vp, sz = ctypes.c_void_p, ctypes.c_size_t
        L.nk_gemm_create.restype = ctypes.c_int
        L.nk_gemm_create.argtypes = [ctypes.POINTER(Desc), ctypes.POINTER(vp)]
        L.nk_gemm_workspace_bytes.restype = sz
        L.nk_gemm_workspace_bytes.argtypes = [vp]
        L.nk_gemm_run.restype = ctypes.c_int
        L.nk_gemm_run.argtypes = [vp, vp, vp, vp, vp, vp, sz, vp]
        L.nk_gemm_run_static.restype = ctypes.c_int
        L.nk_gemm_run_static.argtypes = [vp, vp, vp, vp, vp, vp]
        L.nk_gemm_run_host.restype = ctypes.c_int
        L.nk_gemm_run_host.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
        L.nk_gemm_selftest_timeout.restype = ctypes.c_int
        L.nk_gemm_selftest_timeout.argtypes = [vp, vp]
        L.nk_gemm_check.restype = ctypes.c_int
        L.nk_gemm_check.argtypes = [vp]
        L.nk_gemm_destroy.restype = ctypes.c_int
        L.nk_gemm_destroy.argtypes = [vp]
        L.nk_status_str.restype = ctypes.c_char_p
        L.nk_status_str.argtypes = [ctypes.c_int]
        L.nk_gemm_kernel_name.restype = ctypes.c_char_p
        L.nk_gemm_kernel_name.argtypes = [vp]
        L.nk_gemm_launches_per_run.restype = ctypes.c_int
        L.nk_gemm_launches_per_run.argtypes = [vp]
        L.nk_gemm_last_cuda_error.restype = ctypes.c_char_p
        L.nk_gemm_last_cuda_error.argtypes = [vp]
        L.nk_quantize_s8.restype = ctypes.c_int
        L.nk_quantize_s8.argtypes = [vp, vp, sz, ctypes.c_float, ctypes.c_int, vp]
        _lib = L
    return _lib


def exported_symbols():
    L = lib()
    return [s for s in EXPORTS if hasattr(L, s)]


def _check(status: int, plan=None):
    if status != 0:
        msg = lib().nk_status_str(status).decode()
        if plan is not None:
            extra = lib().nk_gemm_last_cuda_error(plan).decode()
            if extra:
                msg += f" ({extra})"
        raise NkError(status, msg)


def _ptr(x):
    """Device/host pointer of a torch tensor, an int, or None."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    return x.data_ptr()


class Plan:
    """nk_gemm_create / run / destroy.  Tensors are torch tensors used only for
    their pointers; the caller owns every buffer."""

    def __init__(self, M, N, K, in_dtype=BF16, out_dtype=F32, layout_a=ROW_MAJOR,
                 layout_b=ROW_MAJOR, epilogue=EPI_NONE, device=0, flags=0, beta=0, batch=0,
                 stride_a=0, stride_b=0, stride_c=0, batch_independent=0,
                 layout_c=ROW_MAJOR, scale=0.0):
        self.desc = Desc(M, N, K, in_dtype, out_dtype, layout_a, layout_b, epilogue, device, flags,
                         beta, batch, stride_a, stride_b, stride_c, batch_independent, layout_c, scale)
        self._h = ctypes.c_void_p()
        _check(lib().nk_gemm_create(ctypes.byref(self.desc), ctypes.byref(self._h)))

    @property
    def workspace_bytes(self) -> int:
        return lib().nk_gemm_workspace_bytes(self._h)

    @property
    def kernel_name(self) -> str:
        return lib().nk_gemm_kernel_name(self._h).decode()

    @property
    def launches_per_run(self) -> int:
        return lib().nk_gemm_launches_per_run(self._h)

    def run(self, A, B, C, bias=None, workspace=None, workspace_bytes=None, stream=None):
        if workspace_bytes is None:
            workspace_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
        _check(lib().nk_gemm_run(self._h, _ptr(A), _ptr(B), _ptr(bias), _ptr(C), _ptr(workspace),
                                 workspace_bytes, stream), self._h)

    def run_static(self, A, B, C, bias=None, stream=None):
        """nk_gemm_run_static: same GEMM, scratch taken from the library's built-in
        16 MiB device array, so the caller allocates nothing."""
        _check(lib().nk_gemm_run_static(self._h, _ptr(A), _ptr(B), _ptr(bias), _ptr(C), stream), self._h)

    def run_host(self, hA, hB, hC, dA, dB, dC, hbias=None, dbias=None, workspace=None,
                 workspace_bytes=None, stream=None):
        if workspace_bytes is None:
            workspace_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
        _check(lib().nk_gemm_run_host(self._h, _ptr(hA), _ptr(hB), _ptr(hbias), _ptr(hC), _ptr(dA),
                                      _ptr(dB), _ptr(dbias), _ptr(dC), _ptr(workspace),
                                      workspace_bytes, stream), self._h)

    def selftest_timeout(self, stream=None):
        _check(lib().nk_gemm_selftest_timeout(self._h, stream), self._h)

    def check(self):
        _check(lib().nk_gemm_check(self._h), self._h)

    def destroy(self):
        if self._h:
            lib().nk_gemm_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


def quantize_s8(x, q, n, inv_scale, device=0, stream=None):
    """nk_quantize_s8: FP32 device values -> INT8 (round half to even of x * inv_scale, saturating)."""
    _check(lib().nk_quantize_s8(_ptr(x), _ptr(q), n, inv_scale, device, stream))


def plan_for(w, device=0, flags=0) -> Plan:
    """Plan for a workload record with M, N, K, in_dtype ("f32"/"bf16"/"f16"/"s8"), out_dtype,
    layout ("row"/"blocked32") and epilogue ("none"/"bias_relu") attributes."""
    lay_a = BLOCKED32 if w.layout == "blocked32" else ROW_MAJOR
    lay_b = BLOCKED32 if w.layout in ("blocked32", "b_blocked32") else TRANSPOSED if w.layout == "b_transposed" else ROW_MAJOR
    types = {"f32": F32, "bf16": BF16, "f16": F16, "s8": S8, "s32": S32, "e4m3": E4M3, "e5m2": E5M2}
    return Plan(w.M, w.N, w.K, in_dtype=types[w.in_dtype], out_dtype=types[w.out_dtype],
                layout_a=lay_a, layout_b=lay_b,
                epilogue=EPI_BIAS_RELU if w.epilogue == "bias_relu" else EPI_NONE,
                device=device, flags=flags)
