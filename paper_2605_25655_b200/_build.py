"""Builds libthinfer.so in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import shutil
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libthinfer.so")            # IEEE FP16 storage
LIB_BF16 = os.path.join(HERE, "libthinfer_bf16.so")  # BF16 storage: the same sources with -DTHINFER_BF16
VARIANTS = ((LIB, []), (LIB_BF16, ["-DTHINFER_BF16"]))

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a",
    "-lineinfo", "-O3", "-std=c++17",
    "-shared", "-Xcompiler", "-fPIC",
    "--expt-relaxed-constexpr",
]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found: the CUDA extension cannot be built")


def sources():
    return sorted(os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".cu", ".cuh"))) + [
        os.path.join(os.path.dirname(HERE), "include", "thinfer.h")]


def is_stale(lib: str = None) -> bool:
    libs = [lib] if lib else [v[0] for v in VARIANTS]
    for l in libs:
        if not os.path.exists(l):
            return True
        t = os.path.getmtime(l)
        if any(os.path.getmtime(s) > t for s in sources()):
            return True
    return False


def build(force: bool = False, verbose: bool = False) -> str:
    """Compiles every .cu of csrc/ into one shared library per storage type (the two compilations run side by
    side); returns the path of the FP16 library."""
    cus = [s for s in sources() if s.endswith(".cu")]
    extra = os.environ.get("THINFER_NVCC_EXTRA", "").split()
    procs = []
    for lib, defs in VARIANTS:
        if not force and not is_stale(lib):
            continue
        cmd = [_nvcc()] + NVCC_FLAGS + defs + extra + (["-Xptxas", "-v"] if verbose else []) + ["-o", lib] + cus
        procs.append((lib, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
    for lib, p in procs:
        out, _ = p.communicate()
        if p.returncode != 0:
            raise RuntimeError(f"nvcc failed for {os.path.basename(lib)}:\n" + out)
        if verbose:
            print(out)
    return LIB


if __name__ == "__main__":
    import sys
    print(build(force=True, verbose="-v" in sys.argv))
