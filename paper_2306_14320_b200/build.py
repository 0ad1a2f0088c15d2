"""Builds the CUDA shared library (libim2win.so) in-tree with nvcc for sm_100a.

``python -m paper_2306_14320_b200.build`` or ``build_library()``.  nvcc cross-compiles without a GPU.
"""
from __future__ import annotations

import glob
import os
import subprocess
import sys

_HERE = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_HERE)
CSRC = os.path.join(_HERE, "csrc")
LIB = os.path.join(_HERE, "libim2win.so")
ARCH_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a"]


def sources() -> list[str]:
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(_ROOT, "include", "*.h"))
    return any(os.path.getmtime(p) > t for p in deps)


# conv_tc_persistent.cu holds four families of kernel instantiations (by filter size); compiled as
# four translation units (-DIM2WIN_PART=k) they build in parallel.
PARTS = {"conv_tc_persistent.cu": 4}


def build_library(force: bool = False, verbose: bool = False, out: str | None = None,
                  defines: tuple[str, ...] = ()) -> str:
    """Compile every .cu under csrc/ (object files in parallel) into one shared library; returns its
    path.  ``out``/``defines`` build a variant beside the product library (e.g. -DIM2WIN_PROF, the
    wait-cycle counters)."""
    import concurrent.futures
    import shutil
    import tempfile
    target = out or LIB
    if out is None and not (force or _stale()):
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    common = [nvcc, "-std=c++17", "-O3", "-lineinfo", *ARCH_FLAGS, "-Xcompiler", "-fPIC",
              *[f"-D{d}" for d in defines], "-I", os.path.join(_ROOT, "include"), "-I", CSRC]
    if verbose:
        common[1:1] = ["-Xptxas", "-v"]
    objdir = tempfile.mkdtemp(prefix="im2win_build_")
    try:
        jobs = []
        for src in sources():
            base = os.path.basename(src)
            nparts = PARTS.get(base, 0)
            if nparts:
                for k in range(nparts):
                    jobs.append((src, os.path.join(objdir, f"{base}.{k}.o"), [f"-DIM2WIN_PART={k}"]))
            else:
                jobs.append((src, os.path.join(objdir, f"{base}.o"), []))

        def compile_one(job):
            src, obj, extra = job
            subprocess.run([*common, *extra, "-c", src, "-o", obj], check=True)
            return obj

        with concurrent.futures.ThreadPoolExecutor(max_workers=min(len(jobs), os.cpu_count() or 4)) as pool:
            objs = list(pool.map(compile_one, jobs))
        tmp = target + f".tmp{os.getpid()}"
        subprocess.run([nvcc, *ARCH_FLAGS, "-shared", "-o", tmp, *objs], check=True)
        os.replace(tmp, target)
    finally:
        shutil.rmtree(objdir, ignore_errors=True)
    return target


if __name__ == "__main__":
    print(build_library(force="--force" in sys.argv, verbose="-v" in sys.argv))
