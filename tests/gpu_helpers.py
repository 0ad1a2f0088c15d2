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
    ws = Guarded(b.workspace_bytes(dims) // 4) if src_kind in (b.SRC_NCHW, b.SRC_NCHW_FUSED) else None
    b.conv(xd, src_kind, fd, dims, mode, out.view, None if ws is None else ws.view,
           0 if ws is None else ws.n * 4)
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
