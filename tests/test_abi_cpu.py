"""CPU-only checks of the boundary: the shared library loads, exports every
function include/nk_gemm.h declares, validates descriptors before touching a
device, and the Python binding mirrors the header's constants."""
import ctypes
import os
import re

import pytest

import paper_2511_13764_b200 as nk
from paper_2511_13764_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "nk_gemm.h")


def _declared_functions():
    src = open(HEADER).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(nk_[a-z0-9_]+)\s*\(", src)))


def test_library_exports_every_declared_symbol():
    L = ctypes.CDLL(nk.lib_path()) if os.path.exists(nk.lib_path()) else nk.lib()
    names = _declared_functions()
    assert "nk_gemm_create" in names and "nk_gemm_run" in names and "nk_gemm_destroy" in names
    for n in names:
        assert hasattr(L, n), f"{n} declared in nk_gemm.h but not exported"
    assert sorted(binding.EXPORTS) == names


def test_header_constants_match_binding():
    src = open(HEADER).read()
    assert re.search(r"NK_F32\s*=\s*0,\s*NK_BF16\s*=\s*1", src)
    assert re.search(r"NK_ROW_MAJOR\s*=\s*0,\s*NK_BLOCKED32\s*=\s*1", src)
    assert re.search(r"NK_EPI_NONE\s*=\s*0,\s*NK_EPI_BIAS_RELU\s*=\s*1", src)
    assert (nk.F32, nk.BF16, nk.ROW_MAJOR, nk.BLOCKED32, nk.EPI_NONE, nk.EPI_BIAS_RELU) == (0, 1, 0, 1, 0, 1)
    assert "NK_FLAG_SPLITK_SHIFT 8" in src and nk.flag_splitk(3) == 3 << 8
    assert "NK_FLAG_TILE_N_SHIFT 16" in src and nk.flag_tile_n(4) == 4 << 16


def test_status_strings():
    L = nk.lib()
    seen = {L.nk_status_str(i).decode() for i in range(8)}
    assert len(seen) == 8 and "ok" in seen
    assert L.nk_status_str(99).decode() == "unknown status"


@pytest.mark.parametrize("kw,status", [
    (dict(M=0, N=8, K=8), 1),
    (dict(M=8, N=-1, K=8), 1),
    (dict(M=8, N=8, K=8, in_dtype=7), 1),
    (dict(M=8, N=8, K=8, in_dtype=0, out_dtype=1), 1),          # BF16 C needs BF16 inputs
    (dict(M=32, N=32, K=32, in_dtype=0, layout_a=1), 2),        # blocked needs BF16
    (dict(M=48, N=32, K=32, in_dtype=1, layout_a=1), 3),        # blocked needs multiples of 32
    (dict(M=32, N=32, K=48, in_dtype=1, layout_b=1), 3),
    (dict(M=8, N=12, K=8, in_dtype=1), 3),                       # BF16 rows must be 16-byte multiples
    (dict(M=8, N=8, K=6, in_dtype=0), 3),
    (dict(M=32, N=32, K=32, in_dtype=1, layout_a=1, batch=2, stride_a=1028), 3),   # blocked items: strides in 8-element steps too
    (dict(M=32, N=32, K=32, in_dtype=3, out_dtype=4, layout_b=1, batch=2), 2),     # no batch with 8-bit operands
    (dict(M=8, N=8, K=8, in_dtype=1, batch=2, stride_a=68), 3),           # stride not a multiple of 8
    (dict(M=8, N=8, K=8, in_dtype=0, batch=2, stride_b=32), 1),           # items overlap
    (dict(M=8, N=8, K=8, in_dtype=0, beta=2), 1),
    (dict(M=32, N=32, K=32, in_dtype=0, layout_c=1), 2),                 # blocked C needs BF16 operands
    (dict(M=32, N=40, K=32, in_dtype=1, layout_c=1), 3),
    (dict(M=8, N=8, K=8, in_dtype=1, flags=nk.FLAG_KERNEL_SIMT), 2),
    (dict(M=8, N=8, K=8, in_dtype=0, flags=nk.FLAG_KERNEL_UMMA), 2),
])
def test_descriptor_validation_needs_no_device(kw, status):
    with pytest.raises(nk.NkError) as e:
        nk.Plan(**kw)
    assert e.value.status == status


def test_null_arguments():
    L = nk.lib()
    h = ctypes.c_void_p()
    assert L.nk_gemm_create(None, ctypes.byref(h)) == 1
    assert L.nk_gemm_create(ctypes.byref(binding.Desc(8, 8, 8, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0)), None) == 1
    assert L.nk_gemm_destroy(None) == 0
    assert L.nk_gemm_workspace_bytes(None) == 0
    assert L.nk_gemm_run(None, None, None, None, None, None, 0, None) == 1
    assert L.nk_gemm_check(None) == 1
    assert L.nk_gemm_kernel_name(None) == b""


def test_no_cpu_fallback_without_device():
    """On a box without a GPU a valid descriptor is refused with NK_ERR_DEVICE."""
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(nk.NkError) as e:
        nk.Plan(256, 256, 256, nk.F32, nk.F32)
    assert e.value.status == 5


def test_product_never_imports_the_oracle():
    pkg = os.path.join(ROOT, "paper_2511_13764_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.lower(), f"{f} mentions the oracle"
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith((".py", ".c")):
            text = open(os.path.join(ROOT, "oracle", f)).read()
            assert "paper_2511_13764_b200" not in text and "nk_gemm.h" not in text
