"""Builds ``csrc/libllmem.so`` with nvcc for sm_100a (in-tree, no JIT cache)."""
from __future__ import annotations

import os
import shutil
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

_HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_HERE, "csrc")
LIB = os.path.join(CSRC, "libllmem.so")
DEBUG_LIB = os.path.join(CSRC, "libllmem_debug.so")
SOURCES = ("api.cu", "estimate.cu", "events.cu", "scan.cu", "fused.cu")
HEADERS = ("llmem_model.cuh", "llmem_host.h", "fold.cuh", "expand.cuh", "ranges.cuh", "spans.cuh", os.path.join("..", "..", "include", "llmem.h"))

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC", "-Xptxas", "-v",
]


def _nvcc() -> str:
    nvcc = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(nvcc):
        raise RuntimeError("nvcc not found; the CUDA library cannot be built")
    return nvcc


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, s) for s in SOURCES + HEADERS]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, extra_flags=(), out: str | None = None) -> str:
    """Compile every translation unit for sm_100a and link the shared library.
    `extra_flags` (e.g. -D overrides of launch shapes) and `out` serve tuning sweeps."""
    target = out or LIB
    if not force and out is None and not _stale():
        return LIB
    nvcc = _nvcc()
    objdir = os.path.join(CSRC, "_build") if out is None else target + ".objs"
    os.makedirs(objdir, exist_ok=True)

    def compile_one(src: str) -> str:
        obj = os.path.join(objdir, src.replace(".cu", ".o"))
        cmd = [nvcc, *NVCC_FLAGS, *extra_flags, "-c", os.path.join(CSRC, src), "-o", obj]
        r = subprocess.run(cmd, capture_output=True, text=True)
        if verbose or r.returncode != 0:
            sys.stderr.write(r.stdout + r.stderr)
        if r.returncode != 0:
            raise RuntimeError(f"nvcc failed on {src}")
        return obj

    with ThreadPoolExecutor(max_workers=len(SOURCES)) as ex:
        objs = list(ex.map(compile_one, SOURCES))
    tmp = target + f".tmp{os.getpid()}"
    subprocess.check_call([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-shared", "-o", tmp, *objs,
                           "-cudart", "static"])
    os.replace(tmp, target)
    return target


def build_checked(verbose: bool = False) -> str:
    """The same library with -DLLMEM_DEBUG: every index the streaming kernels derive is tested
    before use (csrc/libllmem_debug.so; load it by setting LLMEM_CHECKED=1)."""
    return build(force=True, verbose=verbose, extra_flags=["-DLLMEM_DEBUG"], out=DEBUG_LIB)


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose=True))
