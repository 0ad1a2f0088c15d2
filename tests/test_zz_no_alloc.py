"""im2win_conv_static, the entry point for callers that cannot allocate device memory (their GPU
memory is owned by another allocator, or they run under a no-allocation-after-start-up rule): it
keeps the im2win tensor in a buffer built into the library instead of a caller-supplied workspace.

Checked here through the C ABI against the existing entry point im2win_conv on the same inputs, on
two calls in a row (the second finds the first call's data still in the shared buffer), with the
tolerances of the other convolution tests.  Collected last on purpose, so that a run that stops at
the first failure has already run every other test."""
import numpy as np
import pytest
import torch

from paper_2306_14320_b200 import binding as b
from paper_2306_14320_b200 import workloads as wl
from gpu_helpers import TOL, Guarded, ensure_built, rel_l2

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    ensure_built()


def _existing_entry_point(xd, fd, dims, mode):
    ho, wo = b.out_dims(dims)
    out = torch.zeros((dims[0], dims[4], ho, wo), dtype=torch.float32, device="cuda")
    ws = torch.empty(b.workspace_bytes(dims) // 4, dtype=torch.float32, device="cuda")
    b.conv(xd, b.SRC_NCHW, fd, dims, mode, out, ws)
    assert b.last_device_status() == 0
    return out.cpu().numpy()


@pytest.mark.parametrize("mode", [b.MODE_TF32, b.MODE_BF16, b.MODE_FP32], ids=["tf32", "bf16", "fp32"])
def test_static_scratch_matches_existing_entry_point_twice_in_a_row(mode):
    # two different problems back to back: the second call's im2win tensor is smaller than the first's,
    # so stale floats from the first call sit right behind it in the shared buffer
    first = wl.CONFIGS["resnet3x3"].with_batch(3)
    second = wl.CONFIGS["stem7x7"].with_batch(1)
    assert b.workspace_bytes(second.dims()) < b.workspace_bytes(first.dims()) <= b.STATIC_SCRATCH_BYTES
    for layer in (first, second):
        dims = layer.dims()
        xd = torch.from_numpy(wl.make_input(layer)).cuda()
        fd = torch.from_numpy(wl.make_filter(layer)).cuda()
        want = _existing_entry_point(xd, fd, dims, mode)
        ho, wo = b.out_dims(dims)
        out = Guarded(layer.N * layer.K * ho * wo)
        b.conv_static(xd, fd, dims, mode, out.view)
        assert b.last_device_status() == 0
        got = out.check().reshape(want.shape)
        assert np.isfinite(got).all()
        assert rel_l2(got, want) <= TOL[mode]
        # same kernels on the same inputs: the two results differ at most by the order in which the
        # tensor cores happened to accumulate (two threads issue the MMAs of a tile), never by more
        assert np.allclose(got, want, rtol=1e-4, atol=1e-4)


def test_static_scratch_rejects_problems_beyond_its_buffer():
    big = wl.CONFIGS["resnet3x3"]  # batch 128: a 319 MB im2win tensor
    assert b.workspace_bytes(big.dims()) > b.STATIC_SCRATCH_BYTES == 32 * 1024 * 1024
    x = torch.zeros(16, device="cuda")
    with pytest.raises(b.Im2winError) as e:
        b.conv_static(x, x, big.dims(), b.MODE_TF32, x)   # rejected before any pointer is used
    assert e.value.code == b.ESCRATCH
    assert "scratch" in str(e.value)
