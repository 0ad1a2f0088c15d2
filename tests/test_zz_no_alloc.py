"""im2win_conv_static, the entry point for callers that cannot allocate device memory (their GPU
memory is owned by another allocator, or they run under a no-allocation-after-start-up rule): it
keeps the im2win tensor -- and, behind it, the filter copy some kernels want -- in a buffer built
into the library instead of a caller-supplied workspace.

Checked here through the C ABI on two calls in a row (the second finds the first call's data still
in the shared buffer): against the existing entry point im2win_conv on the same inputs with the
tolerances of the other convolution tests, against the CPU oracle (Eq. 1) itself, bit for bit on
exactly representable data, and for the claim that the call takes no device memory.  Collected last
on purpose, so that a run that stops at the first failure has already run every other test."""
import numpy as np
import pytest
import torch

from paper_2306_14320_b200 import binding as b
from paper_2306_14320_b200 import workloads as wl
from gpu_helpers import TOL, Guarded, ensure_built, oracle_conv, rel_l2

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    ensure_built()
    b.use_test_library(False)  # the product library


def _existing_entry_point(xd, fd, dims, mode):
    ho, wo = b.out_dims(dims)
    out = torch.zeros((dims[0], dims[4], ho, wo), dtype=torch.float32, device="cuda")
    ws = torch.empty(b.conv_workspace_bytes(dims, b.SRC_NCHW, mode) // 4, dtype=torch.float32, device="cuda")
    b.conv(xd, b.SRC_NCHW, fd, dims, mode, out, ws)
    assert b.last_device_status() == 0
    return out.cpu().numpy()


def _static(xd, fd, dims, mode):
    ho, wo = b.out_dims(dims)
    out = Guarded(dims[0] * dims[4] * ho * wo)
    b.conv_static(xd, fd, dims, mode, out.view)
    assert b.last_device_status() == 0
    return out.check().reshape(dims[0], dims[4], ho, wo)


@pytest.mark.parametrize("mode", [b.MODE_TF32, b.MODE_BF16, b.MODE_FP32], ids=["tf32", "bf16", "fp32"])
def test_static_scratch_matches_existing_entry_point_twice_in_a_row(mode):
    # two different problems back to back: the second call's im2win tensor is smaller than the first's,
    # so stale floats from the first call sit right behind it in the shared buffer
    first = wl.CONFIGS["resnet3x3"].with_batch(3)
    second = wl.CONFIGS["stem7x7"].with_batch(1)
    assert b.workspace_bytes(second.dims()) < b.workspace_bytes(first.dims()) <= b.STATIC_SCRATCH_BYTES
    for layer in (first, second):
        dims = layer.dims()
        x, f = wl.make_input(layer), wl.make_filter(layer)
        xd, fd = torch.from_numpy(x).cuda(), torch.from_numpy(f).cuda()
        want = _existing_entry_point(xd, fd, dims, mode)
        got = _static(xd, fd, dims, mode)
        assert np.isfinite(got).all()
        assert rel_l2(got, want) <= TOL[mode]
        # same kernels on the same inputs: the two results differ at most by the order in which the
        # tensor cores happened to accumulate, never by more
        assert np.allclose(got, want, rtol=1e-4, atol=1e-4)
        # and against the oracle itself
        assert rel_l2(got, oracle_conv(x, f, dims)) <= TOL[mode]


# shapes whose filter is too large to stay in shared memory (K > 256; a wide 7x7 layer with 64 channels;
# a deep 3x3 layer): the kernels that stream the filter want a copy of it, which must come out of the
# built-in buffer, never out of an allocation
STREAMED = [(1, 24, 20, 21, 300, 3, 3, 1), (1, 64, 21, 230, 64, 7, 7, 2), (2, 256, 16, 16, 256, 3, 3, 1)]


@pytest.mark.parametrize("mode", [b.MODE_TF32, b.MODE_BF16], ids=["tf32", "bf16"])
@pytest.mark.parametrize("dims", STREAMED + [wl.CONFIGS["resnet3x3"].with_batch(3).dims()])
def test_static_scratch_small_integers_equal_the_oracle_bit_for_bit(dims, mode):
    n, c, h, w, k, fh, fw, s = dims
    x = wl.small_ints(31, n * c * h * w).reshape(n, c, h, w)
    f = wl.small_ints(32, k * c * fh * fw, -2, 2).reshape(k, c, fh, fw)
    xd, fd = torch.from_numpy(x).cuda(), torch.from_numpy(f).cuda()
    ref = oracle_conv(x, f, dims)
    for _ in range(2):
        assert np.array_equal(_static(xd, fd, dims, mode).astype(np.float64), ref)


@pytest.mark.parametrize("mode", [b.MODE_TF32, b.MODE_BF16], ids=["tf32", "bf16"])
@pytest.mark.parametrize("dims", STREAMED + [wl.CONFIGS["stem7x7"].with_batch(1).dims()])
def test_static_scratch_takes_no_device_memory(dims, mode):
    """Free device memory (the driver's figure, which sees every kind of allocation, pools included)
    is the same before and after a second and a third call; the first call may load kernels."""
    n, c, h, w, k, fh, fw, s = dims
    x = wl.normal01(41, n * c * h * w).reshape(n, c, h, w)
    f = (wl.normal01(42, k * c * fh * fw) * np.float32(np.sqrt(2.0 / (c * fh * fw)))).reshape(k, c, fh, fw)
    xd, fd = torch.from_numpy(x).cuda(), torch.from_numpy(f).cuda()
    ho, wo = b.out_dims(dims)
    out = torch.empty((n, k, ho, wo), dtype=torch.float32, device="cuda")
    b.conv_static(xd, fd, dims, mode, out)  # warm-up: module load, first-call set-up
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    for _ in range(2):
        b.conv_static(xd, fd, dims, mode, out)
        torch.cuda.synchronize()
        free1, _ = torch.cuda.mem_get_info()
        assert free1 == free0, (free0, free1)
    assert b.last_device_status() == 0
    assert rel_l2(out.cpu().numpy(), oracle_conv(x, f, dims)) <= TOL[mode]


def test_static_scratch_rejects_problems_beyond_its_buffer():
    big = wl.CONFIGS["resnet3x3"]  # batch 128: a 319 MB im2win tensor
    assert b.workspace_bytes(big.dims()) > b.STATIC_SCRATCH_BYTES == 32 * 1024 * 1024
    x = torch.zeros(16, device="cuda")
    with pytest.raises(b.Im2winError) as e:
        b.conv_static(x, x, big.dims(), b.MODE_TF32, x)   # rejected before any pointer is used
    assert e.value.code == b.ESCRATCH
    assert "scratch" in str(e.value)
