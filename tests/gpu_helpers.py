"""Helpers for the GPU parity tests: run the CUDA path through the C-ABI binding on tensors with guard
bands, and compare with the CPU oracle."""
import numpy as np
import torch

import oracle
from paper_2306_14320_b200 import binding as b
from paper_2306_14320_b200 import build

GUARD = 1024  # floats of sentinel before and after every output buffer
SENTINEL = -7.0e37

TOL = {b.MODE_TF32: 5e-3, b.MODE_BF16: 2e-2, b.MODE_FP32: 2e-6}


def ensure_built():
    build.build_library()


# Kernel configurations of the convolution parity tests.  "auto" and "minws" run the PRODUCT library
# (its own choice of kernel; "minws" with the smallest legal workspace, i.e. without scratch for a
# filter copy); every other one runs the test build of the same code with one diagnostic switch set.
CONV_CONFIGS = {
    "auto": {}, "minws": {},
    "strip": {"force_strip": 1, "strip_pair": 2, "strip_mh": 1, "no_window": 1},
    "strip2": {"force_strip": 1, "strip_pair": 2, "strip_mh": 2, "no_window": 1},
    "pair": {"force_strip": 1, "strip_pair": 1, "strip_mh": 1, "no_window": 1},
    "pair2": {"force_strip": 1, "strip_pair": 1, "strip_mh": 2, "no_window": 1},
    "window": {"force_window": 1}, "window1": {"force_window": 1, "window_mh": 1, "window_pair": 2},
    "window2": {"force_window": 1, "window_mh": 2, "window_pair": 2},
    "wtwo": {"force_window": 1, "window_pair": 2, "window_two": 1},
    "wstream": {"force_window": 1, "window_pair": 2, "window_bres": 2},
    "wpair": {"force_window": 1, "window_mh": 1, "window_pair": 1}, "wpair2": {"force_window": 1, "window_mh": 2, "window_pair": 1},
    "nostrip": {"no_strip": 1, "no_window": 1},
    "nobox": {"no_strip": 1, "no_window": 1, "no_box": 1}, "nopim": {"no_strip": 1, "no_window": 1, "no_pim": 1},
    "split3": {"no_strip": 1, "no_window": 1, "splitk": 3}, "bslice": {"no_strip": 1, "no_window": 1, "bslice": 1},
    "generic": {"force_generic": 1},
}
_KNOB_DEFAULTS = {"force_generic": 0, "no_strip": 0, "force_strip": 0, "no_box": 0, "no_pim": 0, "bslice": 0,
                  "no_bslice": 0, "splitk": -1, "force_stream": 0, "nsets": 0, "no_l2ahead": 0, "no_btma": 0,
                  "ntiles": 0, "transform_gather": 0, "test_skip_copy": 0, "strip_mh": 0, "strip_pair": 0,
                  "force_window": 0, "no_window": 0, "window_mh": 0, "window_plan": 0, "window_pair": 0, "window_two": 0, "window_nohelp": 0, "window_bres": 0, "transform_budget_kb": 0}
_min_workspace = False


def apply_config(name: str = "auto", **extra) -> None:
    """Selects the library (product or test build) and sets the switches of configuration `name`."""
    global _min_workspace
    knobs = dict(CONV_CONFIGS.get(name, {}), **extra)
    _min_workspace = name == "minws"
    b.use_test_library(bool(knobs))
    if knobs:
        for k, v in _KNOB_DEFAULTS.items():
            b.set_option(k, knobs.get(k, v))


def reset_config() -> None:
    global _min_workspace
    _min_workspace = False
    b.use_test_library(True)
    for k, v in _KNOB_DEFAULTS.items():
        b.set_option(k, v)
    b.use_test_library(False)


def conv_workspace_floats(dims, src_kind: int, mode: int) -> int:
    """Workspace the tests hand to im2win_conv: what im2win_conv_workspace_bytes asks for (room for
    the im2win tensor in every case, so that the documented fallbacks can run), or in the "minws"
    configuration only the im2win tensor."""
    least = b.workspace_bytes(dims)
    if _min_workspace:
        return least // 4
    return max(least, b.conv_workspace_bytes(dims, b.SRC_NCHW, mode), b.conv_workspace_bytes(dims, src_kind, mode)) // 4


class Guarded:
    """A device buffer of n floats with sentinel-filled guard bands on both sides; the payload is
    pre-filled with the sentinel too, so elements a kernel forgets to write are seen."""

    def __init__(self, n: int):
        self.n = n
        self.full = torch.full((n + 2 * GUARD,), SENTINEL, dtype=torch.float32, device="cuda")
        self.view = self.full[GUARD:GUARD + n]
        assert self.view.data_ptr() % 16 == 0

    def check(self) -> np.ndarray:
        host = self.full.cpu().numpy()
        assert np.all(host[:GUARD] == np.float32(SENTINEL)), "write before the buffer"
        assert np.all(host[GUARD + self.n:] == np.float32(SENTINEL)), "write past the buffer"
        return host[GUARD:GUARD + self.n]


def gpu_transform(x: np.ndarray, dims) -> np.ndarray:
    xd = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).cuda()
    out = Guarded(b.workspace_bytes(dims) // 4)
    b.transform(xd, dims, out.view)
    assert b.last_device_status() == 0
    return out.check()


def gpu_conv(x: np.ndarray, f: np.ndarray, dims, mode: int, src_kind: int = b.SRC_NCHW) -> np.ndarray:
    """src_kind NCHW: x is the raw input and the call transforms into a workspace; IM2WIN: x is already
    an im2win tensor."""
    n, c, h, w, k, fh, fw, s = dims
    ho, wo = b.out_dims(dims)
    xd = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).cuda()
    fd = torch.from_numpy(np.ascontiguousarray(f, dtype=np.float32)).cuda()
    out = Guarded(n * k * ho * wo)
    ws = Guarded(conv_workspace_floats(dims, src_kind, mode))
    b.conv(xd, src_kind, fd, dims, mode, out.view, ws.view, ws.n * 4)
    status = b.last_device_status()
    assert status == 0, f"device status {status}"
    if ws is not None:
        ws.check()
    return out.check().reshape(n, k, ho, wo)


def rel_l2(got: np.ndarray, ref: np.ndarray) -> float:
    got, ref = got.astype(np.float64).ravel(), ref.astype(np.float64).ravel()
    return float(np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-300))


def oracle_conv(x, f, dims) -> np.ndarray:
    return oracle.conv_direct(x, f, oracle.Shape(*dims))
