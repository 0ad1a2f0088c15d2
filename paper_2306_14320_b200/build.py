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
# The same objects linked with api.cu compiled -DIM2WIN_TEST_KNOBS: the diagnostic switches become
# settable (im2win_debug_set_option).  Only the parity tests load it; the product library reads no switch.
TEST_LIB = os.path.join(_HERE, "libim2win_test.so")
KNOB_SOURCES = ("api.cu",)
ARCH_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a"]


def sources() -> list[str]:
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _stale() -> bool:
    if not os.path.exists(LIB) or not os.path.exists(TEST_LIB):
        return True
    t = min(os.path.getmtime(LIB), os.path.getmtime(TEST_LIB))
    deps = sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(_ROOT, "include", "*.h"))
    return any(os.path.getmtime(p) > t for p in deps)


# conv_tc_persistent.cu holds four families of kernel instantiations (by filter size); compiled as
# four translation units (-DIM2WIN_PART=k) they build in parallel.
PARTS = {"conv_tc_persistent.cu": 8}


def build_library(force: bool = False, verbose: bool = False, out: str | None = None,
                  defines: tuple[str, ...] = ()) -> str:
    """Compile every .cu under csrc/ (object files in parallel) into the product library and, from
    the same objects plus a second compilation of the sources that hold the diagnostic switches, the
    test library; returns the product library's path.  ``out``/``defines`` build one variant beside
    them instead (e.g. -DIM2WIN_PROF, the wait-cycle counters)."""
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

        knob_jobs = []
        if out is None:
            for src in sources():
                if os.path.basename(src) in KNOB_SOURCES:
                    knob_jobs.append((src, os.path.join(objdir, os.path.basename(src) + ".knobs.o"), ["-DIM2WIN_TEST_KNOBS"]))
        with concurrent.futures.ThreadPoolExecutor(max_workers=min(len(jobs) + len(knob_jobs), os.cpu_count() or 4)) as pool:
            all_objs = list(pool.map(compile_one, jobs + knob_jobs))
        objs, knob_objs = all_objs[:len(jobs)], all_objs[len(jobs):]

        def link(objects, dest):
            tmp = dest + f".tmp{os.getpid()}"
            subprocess.run([nvcc, *ARCH_FLAGS, "-shared", "-o", tmp, *objects], check=True)
            os.replace(tmp, dest)

        link(objs, target)
        if out is None:
            swapped = {os.path.join(objdir, os.path.basename(s) + ".o") for s, _, _ in knob_jobs}
            link([o for o in objs if o not in swapped] + knob_objs, TEST_LIB)
    finally:
        shutil.rmtree(objdir, ignore_errors=True)
    return target


if __name__ == "__main__":
    print(build_library(force="--force" in sys.argv, verbose="-v" in sys.argv))
