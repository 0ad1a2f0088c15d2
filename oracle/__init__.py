"""ctypes front end of the CPU oracle (``im2win_oracle.cpp``).

TEST INFRASTRUCTURE ONLY.  Nothing on the product path may import this package;
it exists so that the tests, the smoke check and the benchmark's CPU-baseline leg
can call the plain C++ restatement of the paper's definitions (Eq. 1,
Algorithm 1, Algorithm 2, Section II-B) on numpy arrays.  It imports neither the
CUDA package nor torch.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "im2win_oracle.cpp")
_HDR = os.path.join(_HERE, "im2win_oracle.h")
_LIB = os.path.join(_HERE, "libim2win_oracle.so")


class _Shape(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("N", "C", "H", "W", "K", "Fh", "Fw", "s")]


@dataclass(frozen=True)
class Shape:
    """Problem sizes in the paper's notation (Section II-A): input N x C x H x W,
    filter K x C x Fh x Fw, stride s."""
    N: int
    C: int
    H: int
    W: int
    K: int
    Fh: int
    Fw: int
    s: int

    def _c(self) -> _Shape:
        return _Shape(self.N, self.C, self.H, self.W, self.K, self.Fh, self.Fw, self.s)


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (-O2, OpenMP) if the shared object is missing or stale."""
    stale = (not os.path.exists(_LIB)
             or os.path.getmtime(_LIB) < max(os.path.getmtime(_SRC), os.path.getmtime(_HDR)))
    if force or stale:
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.run(["g++", "-std=c++17", "-O2", "-fopenmp", "-fPIC", "-shared",
                        "-Wall", "-Wextra", "-o", tmp, _SRC], check=True, cwd=_HERE)
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        P = ctypes.POINTER
        fp, dp, sp = P(ctypes.c_float), P(ctypes.c_double), P(_Shape)
        i32p, i64p = P(ctypes.c_int32), P(ctypes.c_int64)
        lib.oracle_out_dims.argtypes = [sp, i32p, i32p]
        lib.oracle_out_dims.restype = ctypes.c_int
        lib.oracle_counts.argtypes = [sp, i64p, i64p, i64p, i64p]
        lib.oracle_counts.restype = ctypes.c_int
        lib.oracle_im2win.argtypes = [fp, sp, fp]
        lib.oracle_im2win.restype = ctypes.c_int64
        lib.oracle_conv_direct.argtypes = [fp, fp, sp, dp]
        lib.oracle_conv_direct.restype = ctypes.c_int
        lib.oracle_conv_via_im2win.argtypes = [fp, fp, sp, dp]
        lib.oracle_conv_via_im2win.restype = ctypes.c_int
        lib.oracle_conv_via_im2col.argtypes = [fp, fp, sp, dp]
        lib.oracle_conv_via_im2col.restype = ctypes.c_int64
        lib.oracle_conv_direct_points.argtypes = [fp, fp, sp, i32p, ctypes.c_int64, dp]
        lib.oracle_conv_direct_points.restype = ctypes.c_int
        lib.oracle_num_threads.argtypes = []
        lib.oracle_num_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def _f32(a: np.ndarray, n: int, what: str) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=np.float32)
    if a.size != n:
        raise ValueError(f"{what}: expected {n} elements, got {a.size}")
    return a


def _ptr(a: np.ndarray, ct):
    return a.ctypes.data_as(ctypes.POINTER(ct))


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def out_dims(sh: Shape) -> tuple[int, int]:
    ho, wo = ctypes.c_int32(), ctypes.c_int32()
    if _load().oracle_out_dims(ctypes.byref(sh._c()), ctypes.byref(ho), ctypes.byref(wo)) != 0:
        raise ValueError(f"invalid shape {sh}")
    return ho.value, wo.value


def counts(sh: Shape) -> dict:
    v = [ctypes.c_int64() for _ in range(4)]
    if _load().oracle_counts(ctypes.byref(sh._c()), *[ctypes.byref(x) for x in v]) != 0:
        raise ValueError(f"invalid shape {sh}")
    return dict(zip(("input", "im2win", "im2col", "output"), (x.value for x in v)))


def im2win(x: np.ndarray, sh: Shape) -> np.ndarray:
    """Algorithm 1.  Returns the im2win tensor, shape (N, C, Ho, W*Fh), fp32."""
    ho, _ = out_dims(sh)
    x = _f32(x, sh.N * sh.C * sh.H * sh.W, "input")
    out = np.empty((sh.N, sh.C, ho, sh.W * sh.Fh), dtype=np.float32)
    n = _load().oracle_im2win(_ptr(x, ctypes.c_float), ctypes.byref(sh._c()), _ptr(out, ctypes.c_float))
    if n != out.size:
        raise RuntimeError(f"oracle_im2win wrote {n} elements, expected {out.size}")
    return out


def _conv(fn, src: np.ndarray, nsrc: int, f: np.ndarray, sh: Shape):
    ho, wo = out_dims(sh)
    src = _f32(src, nsrc, "source")
    f = _f32(f, sh.K * sh.C * sh.Fh * sh.Fw, "filter")
    out = np.empty((sh.N, sh.K, ho, wo), dtype=np.float64)
    rc = fn(_ptr(src, ctypes.c_float), _ptr(f, ctypes.c_float), ctypes.byref(sh._c()),
            _ptr(out, ctypes.c_double))
    if rc < 0:
        raise RuntimeError("oracle convolution rejected its arguments")
    return out, rc


def conv_direct(x: np.ndarray, f: np.ndarray, sh: Shape) -> np.ndarray:
    """Eq. (1) on the raw input; fp64 result, shape (N, K, Ho, Wo)."""
    return _conv(_load().oracle_conv_direct, x, sh.N * sh.C * sh.H * sh.W, f, sh)[0]


def conv_via_im2win(xhat: np.ndarray, f: np.ndarray, sh: Shape) -> np.ndarray:
    """Algorithm 2 on an im2win tensor; fp64 result."""
    ho, _ = out_dims(sh)
    return _conv(_load().oracle_conv_via_im2win, xhat, sh.N * sh.C * ho * sh.W * sh.Fh, f, sh)[0]


def conv_via_im2col(x: np.ndarray, f: np.ndarray, sh: Shape) -> tuple[np.ndarray, int]:
    """Section II-B im2col + matrix product (tiny inputs).  Returns (result, elements of one image's
    im2col matrix as actually materialised)."""
    out, cnt = _conv(_load().oracle_conv_via_im2col, x, sh.N * sh.C * sh.H * sh.W, f, sh)
    return out, int(cnt)


def conv_direct_points(x: np.ndarray, f: np.ndarray, sh: Shape, idx: np.ndarray) -> np.ndarray:
    """Eq. (1) at the listed (i, j, m, n) output coordinates only."""
    x = _f32(x, sh.N * sh.C * sh.H * sh.W, "input")
    f = _f32(f, sh.K * sh.C * sh.Fh * sh.Fw, "filter")
    idx = np.ascontiguousarray(idx, dtype=np.int32).reshape(-1, 4)
    out = np.empty(idx.shape[0], dtype=np.float64)
    rc = _load().oracle_conv_direct_points(_ptr(x, ctypes.c_float), _ptr(f, ctypes.c_float),
                                           ctypes.byref(sh._c()), _ptr(idx, ctypes.c_int32),
                                           idx.shape[0], _ptr(out, ctypes.c_double))
    if rc != 0:
        raise ValueError("oracle_conv_direct_points rejected its arguments")
    return out
