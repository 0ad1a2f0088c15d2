"""GPU parity, transform: the CUDA im2win transformation must equal the oracle's Algorithm 1 bit for bit."""
import numpy as np
import pytest

import oracle
from paper_2306_14320_b200 import workloads as wl
from gpu_helpers import apply_config, ensure_built, gpu_transform, reset_config

pytestmark = pytest.mark.gpu

SMALL = [
    (1, 1, 4, 4, 1, 2, 2, 1), (2, 3, 7, 9, 4, 3, 3, 1), (1, 2, 9, 8, 3, 2, 3, 1), (2, 2, 8, 11, 2, 3, 2, 2),
    (1, 3, 13, 12, 2, 4, 2, 3), (1, 1, 10, 10, 1, 1, 1, 1), (2, 2, 6, 6, 3, 2, 2, 2), (1, 2, 11, 7, 2, 2, 2, 3),
    (1, 1, 12, 13, 2, 1, 3, 4), (1, 2, 5, 5, 2, 5, 5, 1), (3, 5, 33, 37, 2, 3, 3, 1), (2, 3, 64, 64, 2, 5, 5, 2),
    (1, 2, 130, 1031, 1, 7, 7, 2),     # rows wide enough that one CTA takes only a few output rows
    (1, 1, 30, 5000, 1, 11, 3, 4),     # beyond the staging budget: gather fallback
    (1, 1, 1, 1, 1, 1, 1, 1),
    (3, 50, 11, 11, 2, 2, 2, 4),       # many small planes per CTA, stride larger than the filter
    (2, 700, 9, 9, 2, 3, 3, 1), (4, 300, 15, 15, 2, 3, 3, 1), (2, 130, 16, 16, 2, 3, 3, 2),
]


@pytest.fixture(scope="module", autouse=True)
def _built():
    ensure_built()


@pytest.fixture(params=["auto", "gather"], autouse=True)
def _kernel(request):
    """Every case runs twice: with the product library's own choice of kernel (the TMA tile kernel where
    a job's input and output ranges fit its shared-memory budget), and with the staged-gather kernel
    forced (a switch of the test build of the library)."""
    apply_config("gather" if request.param == "gather" else "auto", **({"transform_gather": 1} if request.param == "gather" else {}))
    yield
    reset_config()


def _bits(a):
    return np.ascontiguousarray(a, dtype=np.float32).view(np.uint32).ravel()


@pytest.mark.parametrize("dims", SMALL)
def test_transform_bit_exact_small(dims):
    n, c, h, w = dims[:4]
    x = wl.normal01(100 + h * w, n * c * h * w).reshape(n, c, h, w)
    # a few special bit patterns must survive the copy unchanged
    flat = x.reshape(-1)
    flat[::97] = np.float32(-0.0)
    flat.view(np.uint32)[5::211] = 0x7FC00001  # a NaN payload
    flat.view(np.uint32)[7::313] = 0x00000001  # a denormal
    ref = oracle.im2win(x, oracle.Shape(*dims))
    assert np.array_equal(_bits(gpu_transform(x, dims)), _bits(ref))


@pytest.mark.parametrize("name,batch", [("tiny", 1), ("resnet3x3", 3), ("stem7x7", 2), ("deep3x3", 3), ("down3x3", 2)]
                         + [(l.name, 2) for l in wl.SWEEP])
def test_transform_bit_exact_layer_shapes(name, batch):
    layer = wl.CONFIGS[name].with_batch(batch)
    x = wl.make_input(layer)
    ref = oracle.im2win(x, oracle.Shape(*layer.dims()))
    assert np.array_equal(_bits(gpu_transform(x, layer.dims())), _bits(ref))


@pytest.mark.parametrize("name", ["resnet3x3", "stem7x7", "deep3x3", "down3x3"])
def test_transform_bit_exact_full_batch(name):
    """The launch configuration the benchmark times (batch 128), every element compared."""
    layer = wl.CONFIGS[name]
    x = wl.make_input(layer)
    ref = oracle.im2win(x, oracle.Shape(*layer.dims()))
    got = gpu_transform(x, layer.dims())
    assert got.size == ref.size
    assert np.array_equal(_bits(got), _bits(ref))


@pytest.mark.parametrize("batch", [32, 128])
@pytest.mark.parametrize("layer", wl.SWEEP, ids=lambda l: l.name)
def test_transform_bit_exact_sweep_layers_batch_32_and_128(layer, batch):
    """The twelve-layer sweep at the batch sizes the benchmark times, every element compared."""
    layer = layer.with_batch(batch)
    x = wl.make_input(layer)
    ref = oracle.im2win(x, oracle.Shape(*layer.dims()))
    got = gpu_transform(x, layer.dims())
    assert got.size == ref.size
    assert np.array_equal(_bits(got), _bits(ref))


def test_bounded_wait_expiry_is_reported_and_the_context_survives(request):
    """Failure detection without a fault: a switch of the test build makes the tile kernel announce its
    input copy but never issue it (single-CTA problem), so the bounded wait runs out after about a
    second.  The kernel must return by itself, the status call must return ETIMEOUT and name the wait,
    and the next call must work."""
    if "gather" in request.node.name:
        pytest.skip("the hook belongs to the tile kernel")
    import time
    import torch
    from paper_2306_14320_b200 import binding as b
    from gpu_helpers import Guarded
    dims = (1, 1, 8, 8, 1, 3, 3, 1)
    x = wl.normal01(77, 64).reshape(1, 1, 8, 8)
    xd = torch.from_numpy(x).cuda()
    out = Guarded(b.workspace_bytes(dims) // 4)
    apply_config("hook", test_skip_copy=1)
    t0 = time.perf_counter()
    b.transform(xd, dims, out.view)
    rc, status = b.last_device_status_rc()  # synchronises the stream
    waited = time.perf_counter() - t0
    b.set_option("test_skip_copy", 0)
    assert rc == b.ETIMEOUT and status == 109, (rc, status)  # DEV_TIMEOUT_COPY
    assert 0.5 < waited < 20.0, waited
    assert b.last_device_status() == 0  # reading the word cleared it
    ref = oracle.im2win(x, oracle.Shape(*dims))
    assert np.array_equal(_bits(gpu_transform(x, dims)), _bits(ref))
