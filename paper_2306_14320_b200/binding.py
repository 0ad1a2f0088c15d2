"""Thin ctypes binding of libim2win.so: same names as the C ABI (include/im2win.h), argument
marshalling only.  Every step of the path runs in the CUDA kernels behind those calls.

torch is used for device memory and streams: tensor arguments are passed as ``data_ptr()`` and the
launch goes to ``torch.cuda.current_stream()``.  There is no fallback of any kind: if the shared
library is missing this module raises at first use, and the launching calls raise ``Im2winError``
when the library reports an error (for example no CUDA device).
"""
from __future__ import annotations

import ctypes
import os
from typing import Sequence

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libim2win.so")
# The same code with settable diagnostic switches (im2win_debug_set_option); loaded by the parity tests
# only, through use_test_library().
TEST_LIB_PATH = os.path.join(_HERE, "libim2win_test.so")

SRC_NCHW, SRC_IM2WIN, SRC_NCHW_FUSED, SRC_IM2WIN_BF16 = 0, 1, 2, 3
MODE_TF32, MODE_BF16, MODE_FP32 = 0, 1, 2
OK, EINVAL, EALIGN, EWORKSPACE, EOVERLAP, ECUDA, ETIMEOUT, EUNSUPPORTED, ESCRATCH = 0, -1, -2, -3, -4, -5, -6, -7, -8

EXPORTS = ("im2win_out_dims", "im2win_workspace_bytes", "im2win_conv_workspace_bytes", "im2win_im2col_bytes", "im2win_transform",
           "im2win_workspace_bytes_bf16", "im2win_transform_bf16", "im2win_conv", "im2win_conv_nhwc", "im2win_conv_bf16out", "im2win_conv_host", "im2win_host_release", "im2win_conv_static",
           "im2win_last_device_status", "im2win_strerror")
STATIC_SCRATCH_BYTES = 32 * 1024 * 1024  # IM2WIN_STATIC_SCRATCH_BYTES of include/im2win.h


class Shape(ctypes.Structure):
    """im2win_shape: N, C, H, W, K, Fh, Fw, stride (all int32)."""
    _fields_ = [(n, ctypes.c_int32) for n in ("N", "C", "H", "W", "K", "Fh", "Fw", "stride")]

    @classmethod
    def of(cls, dims: "Shape | Sequence[int]") -> "Shape":
        return dims if isinstance(dims, cls) else cls(*[int(d) for d in dims])


class Im2winError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {strerror(code)} ({code})")


_lib = None
_test_lib = None
_use_test = False


def _declare(L: ctypes.CDLL) -> ctypes.CDLL:
    sp, vp = ctypes.POINTER(Shape), ctypes.c_void_p
    L.im2win_out_dims.argtypes = [sp, ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_int32)]
    L.im2win_workspace_bytes.argtypes = [sp, ctypes.POINTER(ctypes.c_size_t)]
    L.im2win_conv_workspace_bytes.argtypes = [sp, ctypes.c_int, ctypes.c_int, ctypes.POINTER(ctypes.c_size_t)]
    L.im2win_im2col_bytes.argtypes = [sp, ctypes.POINTER(ctypes.c_size_t)]
    L.im2win_transform.argtypes = [vp, sp, vp, vp]
    L.im2win_workspace_bytes_bf16.argtypes = [sp, ctypes.POINTER(ctypes.c_size_t)]
    L.im2win_transform_bf16.argtypes = [vp, sp, vp, vp]
    L.im2win_conv.argtypes = [vp, ctypes.c_int, vp, sp, ctypes.c_int, vp, vp, ctypes.c_size_t, vp]
    L.im2win_conv_bf16out.argtypes = [vp, ctypes.c_int, vp, sp, ctypes.c_int, vp, vp, ctypes.c_size_t, vp]
    L.im2win_conv_nhwc.argtypes = [vp, ctypes.c_int, vp, sp, ctypes.c_int, vp, vp, ctypes.c_size_t, vp]
    L.im2win_conv_host.argtypes = [vp, vp, sp, ctypes.c_int, vp]
    L.im2win_host_release.argtypes = []
    L.im2win_conv_static.argtypes = [vp, vp, sp, ctypes.c_int, vp, vp]
    L.im2win_last_device_status.argtypes = [vp, ctypes.POINTER(ctypes.c_int32)]
    L.im2win_strerror.argtypes = [ctypes.c_int]
    L.im2win_strerror.restype = ctypes.c_char_p
    for name in EXPORTS[:-1]:
        getattr(L, name).restype = ctypes.c_int
    return L


def lib() -> ctypes.CDLL:
    """Loads libim2win.so (built in-tree by ``paper_2306_14320_b200.build``), or the test build of it
    after use_test_library(True)."""
    global _lib, _test_lib
    path = TEST_LIB_PATH if _use_test else LIB_PATH
    cur = _test_lib if _use_test else _lib
    if cur is None:
        if not os.path.exists(path):
            raise ImportError(f"{path} is missing: build it with `python -m paper_2306_14320_b200.build` "
                              "(there is no non-CUDA fallback)")
        cur = _declare(ctypes.CDLL(path))
        if _use_test:
            cur.im2win_debug_set_option.argtypes = [ctypes.c_char_p, ctypes.c_int]
            cur.im2win_debug_set_option.restype = ctypes.c_int
            cur.im2win_debug_last_kernel.argtypes = []
            cur.im2win_debug_last_kernel.restype = ctypes.c_int
            _test_lib = cur
        else:
            _lib = cur
    return cur


def use_test_library(on: bool) -> None:
    """Route every later call through libim2win_test.so (on) or back through the product library (off).
    The two are separate loaded images: each has its own device status word and built-in buffers."""
    global _use_test
    _use_test = bool(on)


def set_option(name: str, value: int) -> None:
    """Test build only: set one diagnostic switch of the launchers (see Knobs in csrc/common.cuh)."""
    if not _use_test:
        raise RuntimeError("diagnostic switches exist in the test library only: call use_test_library(True) first")
    _check(lib().im2win_debug_set_option(name.encode(), int(value)), f"im2win_debug_set_option({name})")


def _check(code: int, where: str) -> None:
    if code != OK:
        raise Im2winError(code, where)


def _ptr(t) -> int:
    """Device (or host) address of a torch tensor / numpy array / int."""
    if t is None:
        return 0
    if isinstance(t, int):
        return t
    if hasattr(t, "data_ptr"):
        if not t.is_contiguous():
            raise ValueError("tensor must be contiguous")
        return t.data_ptr()
    if hasattr(t, "ctypes"):
        return t.ctypes.data
    raise TypeError(type(t))


def _stream(stream) -> int:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    return int(getattr(stream, "cuda_stream", stream))


def strerror(code: int) -> str:
    return lib().im2win_strerror(int(code)).decode()


def out_dims(shape) -> tuple[int, int]:
    ho, wo = ctypes.c_int32(), ctypes.c_int32()
    _check(lib().im2win_out_dims(ctypes.byref(Shape.of(shape)), ctypes.byref(ho), ctypes.byref(wo)), "im2win_out_dims")
    return ho.value, wo.value


def workspace_bytes(shape) -> int:
    b = ctypes.c_size_t()
    _check(lib().im2win_workspace_bytes(ctypes.byref(Shape.of(shape)), ctypes.byref(b)), "im2win_workspace_bytes")
    return b.value


KERNEL_STRIP, KERNEL_PERSISTENT, KERNEL_GENERIC, KERNEL_FP32, KERNEL_WINDOW = 1, 2, 3, 4, 5


def last_kernel() -> int:
    """Test build only: which convolution kernel the last call launched (KERNEL_*)."""
    if not _use_test:
        raise RuntimeError("the test library only: call use_test_library(True) first")
    return lib().im2win_debug_last_kernel()


def conv_workspace_bytes(shape, src_kind: int, mode: int) -> int:
    """im2win_conv_workspace_bytes: the workspace with which im2win_conv can use its fastest kernel."""
    b = ctypes.c_size_t()
    _check(lib().im2win_conv_workspace_bytes(ctypes.byref(Shape.of(shape)), int(src_kind), int(mode), ctypes.byref(b)),
           "im2win_conv_workspace_bytes")
    return b.value


def im2col_bytes(shape) -> int:
    b = ctypes.c_size_t()
    _check(lib().im2win_im2col_bytes(ctypes.byref(Shape.of(shape)), ctypes.byref(b)), "im2win_im2col_bytes")
    return b.value


def transform(in_nchw, shape, out_im2win, stream=None) -> None:
    """im2win_transform on the current (or given) stream; asynchronous."""
    _check(lib().im2win_transform(_ptr(in_nchw), ctypes.byref(Shape.of(shape)), _ptr(out_im2win), _stream(stream)),
           "im2win_transform")


def workspace_bytes_bf16(shape) -> int:
    b = ctypes.c_size_t()
    _check(lib().im2win_workspace_bytes_bf16(ctypes.byref(Shape.of(shape)), ctypes.byref(b)),
           "im2win_workspace_bytes_bf16")
    return b.value


def transform_bf16(in_nchw, shape, out_im2win_bf16, stream=None) -> None:
    """im2win_transform_bf16 (the im2win tensor stored as bf16) on the current (or given) stream."""
    _check(lib().im2win_transform_bf16(_ptr(in_nchw), ctypes.byref(Shape.of(shape)), _ptr(out_im2win_bf16),
                                       _stream(stream)), "im2win_transform_bf16")


def conv(src, src_kind: int, filter_kcfhfw, shape, mode: int, out_nchw, workspace=None,
         workspace_nbytes: int | None = None, stream=None) -> None:
    """im2win_conv on the current (or given) stream; asynchronous."""
    if workspace_nbytes is None:
        workspace_nbytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(lib().im2win_conv(_ptr(src), int(src_kind), _ptr(filter_kcfhfw), ctypes.byref(Shape.of(shape)),
                             int(mode), _ptr(out_nchw), _ptr(workspace), int(workspace_nbytes), _stream(stream)),
           "im2win_conv")


def conv_nhwc(src, src_kind: int, filter_kcfhfw, shape, mode: int, out_nhwc, workspace=None, workspace_bytes=None,
              stream=None) -> None:
    """im2win_conv_nhwc: like conv(), the fp32 output written N x Ho x Wo x K."""
    if workspace_bytes is None:
        workspace_bytes = workspace.numel() * workspace.element_size() if workspace is not None else 0
    _check(lib().im2win_conv_nhwc(_ptr(src), int(src_kind), _ptr(filter_kcfhfw), ctypes.byref(Shape.of(shape)),
                                  int(mode), _ptr(out_nhwc), _ptr(workspace), int(workspace_bytes),
                                  _stream(stream)), "im2win_conv_nhwc")


def conv_bf16out(src, src_kind: int, filter_kcfhfw, shape, mode: int, out_nchw_bf16, workspace=None,
                 workspace_nbytes: int | None = None, stream=None) -> None:
    """im2win_conv_bf16out: like conv(), the output stored as bf16 (16-bit words)."""
    if workspace_nbytes is None:
        workspace_nbytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(lib().im2win_conv_bf16out(_ptr(src), int(src_kind), _ptr(filter_kcfhfw), ctypes.byref(Shape.of(shape)),
                                     int(mode), _ptr(out_nchw_bf16), _ptr(workspace), int(workspace_nbytes),
                                     _stream(stream)), "im2win_conv_bf16out")


def conv_host(in_host, filter_host, shape, mode: int, out_host) -> None:
    """im2win_conv_host: HOST buffers in, HOST buffer out; returns when the result is there."""
    _check(lib().im2win_conv_host(_ptr(in_host), _ptr(filter_host), ctypes.byref(Shape.of(shape)), int(mode),
                                  _ptr(out_host)), "im2win_conv_host")


def conv_static(in_nchw, filter_kcfhfw, shape, mode: int, out_nchw, stream=None) -> None:
    """im2win_conv_static: like conv() on the untransformed input, but the im2win tensor lives in the
    library's built-in device buffer, so no workspace is passed and nothing is allocated.  For callers
    that cannot allocate device memory.  Raises Im2winError(ESCRATCH) if the problem does not fit.  All
    calls on a device share that buffer: do not let two of them overlap on the GPU."""
    _check(lib().im2win_conv_static(_ptr(in_nchw), _ptr(filter_kcfhfw), ctypes.byref(Shape.of(shape)), int(mode),
                                    _ptr(out_nchw), _stream(stream)), "im2win_conv_static")


def host_release() -> None:
    _check(lib().im2win_host_release(), "im2win_host_release")


def last_device_status_rc(stream=None) -> tuple[int, int]:
    """im2win_last_device_status: (return code, raw status word).  The return code is ETIMEOUT when the
    word names an expired bounded wait, OK otherwise."""
    st = ctypes.c_int32()
    rc = lib().im2win_last_device_status(_stream(stream), ctypes.byref(st))
    if rc not in (OK, ETIMEOUT):
        raise Im2winError(rc, "im2win_last_device_status")
    return rc, st.value


def last_device_status(stream=None) -> int:
    """The raw status word (0 = clean); synchronises the stream and clears the word."""
    return last_device_status_rc(stream)[1]
