"""In-tree build of the CUDA library (nvcc, sm_100a only)."""
from __future__ import annotations

import hashlib
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libnk_gemm.so")
SOURCES = ["nk_gemm.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-shared", "-Xcompiler", "-fPIC"]


STAMP = LIB + ".srchash"


def source_hash() -> str:
    """Hash of everything the library is compiled from (and of the flags): a check-out or a
    copy of the tree may not keep file times, so staleness is decided on contents."""
    h = hashlib.sha256(" ".join(NVCC_FLAGS).encode())
    files = sorted(os.path.join(CSRC, f) for f in os.listdir(CSRC))
    files.append(os.path.join(os.path.dirname(HERE), "include", "nk_gemm.h"))
    for path in files:
        h.update(os.path.basename(path).encode())
        with open(path, "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def _stale() -> bool:
    if not os.path.exists(LIB) or not os.path.exists(STAMP):
        return True
    with open(STAMP) as f:
        return f.read().strip() != source_hash()


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile csrc/*.cu into libnk_gemm.so next to this file (unless it is already built from
    the sources as they are now); returns its path."""
    if not force and not _stale():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    flags = list(NVCC_FLAGS)
    if verbose:
        flags += ["-Xptxas", "-v"]
    tmp = LIB + f".{os.getpid()}.tmp"
    cmd = [nvcc] + flags + ["-o", tmp] + [os.path.join(CSRC, s) for s in SOURCES] + ["-lcudart"]
    subprocess.check_call(cmd)
    os.replace(tmp, LIB)
    with open(STAMP + f".{os.getpid()}.tmp", "w") as f:
        f.write(source_hash())
    os.replace(STAMP + f".{os.getpid()}.tmp", STAMP)
    return LIB


if __name__ == "__main__":
    import sys
    print(build(force=True, verbose="-v" in sys.argv))
