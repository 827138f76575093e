"""nk_gemm: dense GEMM for B200 behind a C ABI.  This package is the thin Python
binding (ctypes marshalling only); all arithmetic runs in the CUDA library."""
from .binding import (  # noqa: F401
    Plan, NkError, lib, lib_path, exported_symbols,
    F32, BF16, F16, S8, S32, E4M3, E5M2, ROW_MAJOR, BLOCKED32, TRANSPOSED, EPI_NONE, EPI_BIAS_RELU,
    FLAG_KERNEL_NAIVE, FLAG_KERNEL_SIMT, FLAG_KERNEL_UMMA, FLAG_REPACK_B, FLAG_SINGLE_CTA, FLAG_CTA_PAIR,
    FLAG_SCALAR_FMA, FLAG_SEPARATE_REDUCE, FLAG_LSU_STORE, FLAG_NO_TAIL_SPLIT, FLAG_F32_TENSOR,
    flag_splitk, flag_tile_n, flag_tail_split, flag_raster, plan_for, quantize_s8, STATIC_SCRATCH_BYTES,
)
