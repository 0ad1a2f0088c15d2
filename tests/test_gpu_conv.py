"""GPU parity, convolution: the CUDA im2win convolution against the oracle's Eq. (1) in double.

Tolerances (relative L2 over the whole output): 5e-3 in TF32 mode, 2e-2 in BF16 mode (the benchmark
definition's), 2e-6 in the fp32 CUDA-core mode.  On small-integer data every product and partial sum
is exact in all modes, so the result must be bit-identical to the oracle: that separates layout
mistakes from rounding."""
import itertools

import numpy as np
import pytest

import oracle
from paper_2306_14320_b200 import binding as b
from paper_2306_14320_b200 import workloads as wl
from gpu_helpers import TOL, ensure_built, gpu_conv, oracle_conv, rel_l2

pytestmark = pytest.mark.gpu

MODES = [b.MODE_FP32, b.MODE_TF32, b.MODE_BF16]
MODE_ID = {b.MODE_FP32: "fp32", b.MODE_TF32: "tf32", b.MODE_BF16: "bf16"}

SMALL = [
    (1, 1, 4, 4, 2, 2, 2, 1), (2, 3, 7, 9, 4, 3, 3, 1), (1, 2, 9, 8, 3, 2, 3, 1), (2, 2, 8, 11, 2, 3, 2, 2),
    (1, 3, 13, 12, 2, 4, 2, 3), (1, 1, 10, 10, 1, 1, 1, 1), (2, 2, 6, 6, 3, 2, 2, 2), (1, 2, 11, 7, 2, 2, 2, 3),
    (1, 1, 12, 13, 2, 1, 3, 4), (3, 2, 5, 5, 2, 5, 5, 1),          # 1x1 outputs: a tile spans many images
    (2, 20, 19, 23, 40, 3, 3, 1),                                     # C, K not multiples of the tile sizes
    (1, 9, 40, 41, 300, 3, 3, 2),                                     # K > 256: two filter tiles
    (5, 7, 9, 9, 17, 3, 3, 1),                                        # 49 positions per image: tiles straddle images
    (2, 3, 37, 35, 24, 7, 7, 2), (1, 3, 51, 51, 32, 11, 11, 4), (1, 12, 14, 14, 16, 5, 5, 1),
    (1, 24, 20, 21, 300, 3, 3, 1),       # streamed filter; in BF16 mode groups of 72 padded to 80 in the bf16 copy
    (1, 16, 21, 230, 16, 7, 7, 2),       # wide 7x7: sixteen-channel strip stages do not fit, eight-channel groups
    (1, 64, 21, 230, 64, 7, 7, 2),       # the same with a filter too large to be resident
]


@pytest.fixture(scope="module", autouse=True)
def _built():
    ensure_built()


@pytest.fixture(params=["auto", "nobox", "nopim", "split3", "bslice", "generic"], autouse=True)
def _kernel(request, monkeypatch):
    """Every case runs six times: with the library's own choice of tensor-core kernel (the persistent,
    filter-size-specialised one where it applies, tiles cut per image and strips staged by 2-D TMA
    boxes where they qualify, reduction slices where its cost model wants them), with the box staging
    switched off (per-image tiles, bulk copies), with per-image tiling switched off as well (tiles
    that span images), with three reduction slices forced wherever a layer has that many channel
    groups (partial sums added into the zeroed output), with the slice-resident filter mode forced
    (every CTA keeps one reduction slice of the filter in shared memory), and with the generic kernel
    forced."""
    monkeypatch.setenv("IM2WIN_FORCE_GENERIC", "1" if request.param == "generic" else "0")
    monkeypatch.setenv("IM2WIN_NO_BOX", "1" if request.param == "nobox" else "0")
    monkeypatch.setenv("IM2WIN_NO_PIM", "1" if request.param == "nopim" else "0")
    monkeypatch.setenv("IM2WIN_BSLICE", "1" if request.param == "bslice" else "0")
    if request.param == "split3":
        monkeypatch.setenv("IM2WIN_SPLITK", "3")
    else:
        monkeypatch.delenv("IM2WIN_SPLITK", raising=False)


def _data(dims, seed, ints=False):
    n, c, h, w, k, fh, fw, s = dims
    if ints:
        x = wl.small_ints(seed, n * c * h * w).reshape(n, c, h, w)
        f = wl.small_ints(seed + 1, k * c * fh * fw, -2, 2).reshape(k, c, fh, fw)
    else:
        x = wl.normal01(seed, n * c * h * w).reshape(n, c, h, w)
        f = (wl.normal01(seed + 1, k * c * fh * fw) * np.float32(np.sqrt(2.0 / (c * fh * fw)))).reshape(k, c, fh, fw)
    return x, f


@pytest.mark.parametrize("mode", MODES, ids=MODE_ID.get)
@pytest.mark.parametrize("dims", SMALL)
def test_conv_small_shapes(dims, mode):
    x, f = _data(dims, 300)
    ref = oracle_conv(x, f, dims)
    got = gpu_conv(x, f, dims, mode)
    assert np.isfinite(got).all()
    assert rel_l2(got, ref) <= TOL[mode]


@pytest.mark.parametrize("mode", [b.MODE_TF32, b.MODE_BF16], ids=MODE_ID.get)
@pytest.mark.parametrize("dims", SMALL + [(3, 16, 30, 30, 32, 3, 3, 1), (2, 32, 21, 25, 24, 5, 5, 1), (3, 8, 20, 22, 40, 3, 3, 2)])
def test_conv_fused_source_small_shapes(dims, mode):
    """src_kind NCHW_FUSED: windows built from staged input rows, no im2win tensor in memory (shapes
    without a fused specialisation take the documented fallback through the workspace)."""
    x, f = _data(dims, 600)
    got = gpu_conv(x, f, dims, mode, src_kind=b.SRC_NCHW_FUSED)
    assert rel_l2(got, oracle_conv(x, f, dims)) <= TOL[mode]
    xi, fi = _data(dims, 700, ints=True)
    assert np.array_equal(gpu_conv(xi, fi, dims, mode, src_kind=b.SRC_NCHW_FUSED).astype(np.float64), oracle_conv(xi, fi, dims))


@pytest.mark.parametrize("mode", [b.MODE_TF32, b.MODE_BF16], ids=MODE_ID.get)
@pytest.mark.parametrize("name,batch", [("tiny", 1), ("resnet3x3", 3), ("stem7x7", 1), ("deep3x3", 3), ("down3x3", 2)]
                         + [(l.name, 1) for l in wl.SWEEP])
def test_conv_fused_source_layer_shapes(name, batch, mode):
    layer = wl.CONFIGS[name].with_batch(batch)
    x, f = wl.make_input(layer), wl.make_filter(layer)
    got = gpu_conv(x, f, layer.dims(), mode, src_kind=b.SRC_NCHW_FUSED)
    assert rel_l2(got, oracle_conv(x, f, layer.dims())) <= TOL[mode]


def test_conv_fused_source_needs_no_workspace(request):
    import torch
    if "generic" in request.node.name:
        pytest.skip("the generic kernel has no fused source; that fallback needs a workspace")
    layer = wl.CONFIGS["resnet3x3"].with_batch(2)
    dims = layer.dims()
    x, f = wl.make_input(layer), wl.make_filter(layer)
    ho, wo = b.out_dims(dims)
    xd, fd = torch.from_numpy(x).cuda(), torch.from_numpy(f).cuda()
    out = torch.zeros((2, layer.K, ho, wo), dtype=torch.float32, device="cuda")
    b.conv(xd, b.SRC_NCHW_FUSED, fd, dims, b.MODE_TF32, out, None, 0)
    assert b.last_device_status() == 0
    assert rel_l2(out.cpu().numpy(), oracle_conv(x, f, dims)) <= TOL[b.MODE_TF32]


@pytest.mark.parametrize("mode", MODES, ids=MODE_ID.get)
@pytest.mark.parametrize("dims", SMALL)
def test_conv_small_integers_bit_exact(dims, mode):
    x, f = _data(dims, 400, ints=True)
    ref = oracle_conv(x, f, dims)
    assert np.abs(ref).max() < 2 ** 24
    got = gpu_conv(x, f, dims, mode)
    assert np.array_equal(got.astype(np.float64), ref)


@pytest.mark.parametrize("mode", [b.MODE_TF32, b.MODE_BF16], ids=MODE_ID.get)
def test_conv_one_hot_filters_are_strided_crops(mode):
    dims = (2, 3, 20, 22, 18, 3, 3, 2)
    n, c, h, w, k, fh, fw, s = dims
    x = wl.small_ints(77, n * c * h * w).reshape(n, c, h, w)
    f = np.zeros((k, c, fh, fw), np.float32)
    taps = list(itertools.product(range(c), range(fh), range(fw)))[:k]
    for j, (r, u, v) in enumerate(taps):
        f[j, r, u, v] = 1.0
    got = gpu_conv(x, f, dims, mode)
    ho, wo = b.out_dims(dims)
    for j, (r, u, v) in enumerate(taps):
        crop = x[:, r, u:u + (ho - 1) * s + 1:s, v:v + (wo - 1) * s + 1:s]
        assert np.array_equal(got[:, j], crop), (j, r, u, v)


@pytest.mark.parametrize("mode", [b.MODE_TF32, b.MODE_BF16], ids=MODE_ID.get)
def test_conv_from_prebuilt_im2win_tensor(mode):
    dims = (2, 16, 30, 30, 32, 3, 3, 1)
    x, f = _data(dims, 500)
    xhat = oracle.im2win(x, oracle.Shape(*dims))
    got = gpu_conv(xhat, f, dims, mode, src_kind=b.SRC_IM2WIN)
    assert rel_l2(got, oracle_conv(x, f, dims)) <= TOL[mode]


@pytest.mark.parametrize("mode", MODES, ids=MODE_ID.get)
@pytest.mark.parametrize("name,batch", [("tiny", 1), ("resnet3x3", 2), ("stem7x7", 1), ("deep3x3", 3), ("down3x3", 1)])
def test_conv_named_configs_reduced_batch(name, batch, mode):
    layer = wl.CONFIGS[name].with_batch(batch)
    x, f = wl.make_input(layer), wl.make_filter(layer)
    ref = oracle_conv(x, f, layer.dims())
    got = gpu_conv(x, f, layer.dims(), mode)
    err = rel_l2(got, ref)
    assert err <= TOL[mode], err
    if mode != b.MODE_FP32:
        # a reduced-precision mode that is "too exact" is not the mode it claims to be
        assert err > 1e-5


@pytest.mark.parametrize("mode", [b.MODE_TF32, b.MODE_BF16], ids=MODE_ID.get)
@pytest.mark.parametrize("layer", wl.SWEEP, ids=lambda l: l.name)
def test_conv_sweep_layers_batch1(layer, mode):
    layer = layer.with_batch(1)
    x, f = wl.make_input(layer), wl.make_filter(layer)
    assert rel_l2(gpu_conv(x, f, layer.dims(), mode), oracle_conv(x, f, layer.dims())) <= TOL[mode]


@pytest.mark.parametrize("mode", [b.MODE_TF32, b.MODE_BF16], ids=MODE_ID.get)
@pytest.mark.parametrize("layer", wl.TABLE_I_LAYERS, ids=lambda l: l.name)
def test_conv_table1_layers_batch1(layer, mode):
    """The paper's own twelve layers (Table I, unpadded), one image each."""
    layer = layer.with_batch(1)
    x, f = wl.make_input(layer), wl.make_filter(layer)
    assert rel_l2(gpu_conv(x, f, layer.dims(), mode), oracle_conv(x, f, layer.dims())) <= TOL[mode]


@pytest.mark.parametrize("mode", [b.MODE_TF32, b.MODE_BF16], ids=MODE_ID.get)
@pytest.mark.parametrize("name", ["resnet3x3", "stem7x7", "deep3x3", "down3x3"])
def test_conv_full_batch_sampled(name, mode):
    """Batch 128, the launch configuration the benchmark times.  The oracle evaluates Eq. (1) at 20000
    sampled output coordinates (plus every corner of the output tensor) and at the whole first and
    last image."""
    layer = wl.CONFIGS[name]
    dims = layer.dims()
    n, c, h, w, k, fh, fw, s = dims
    x, f = wl.make_input(layer), wl.make_filter(layer)
    got = gpu_conv(x, f, dims, mode)
    ho, wo = b.out_dims(dims)
    rng = np.random.default_rng(1234)
    idx = np.stack([rng.integers(0, n, 20000), rng.integers(0, k, 20000), rng.integers(0, ho, 20000),
                    rng.integers(0, wo, 20000)], axis=1).astype(np.int32)
    corners = np.array(list(itertools.product((0, n - 1), (0, k - 1), (0, ho - 1), (0, wo - 1))), dtype=np.int32)
    idx = np.concatenate([idx, corners])
    ref = oracle.conv_direct_points(x, f, oracle.Shape(*dims), idx)
    sample = got[idx[:, 0], idx[:, 1], idx[:, 2], idx[:, 3]]
    assert rel_l2(sample, ref) <= TOL[mode]
    for img in (0, n - 1):
        one = layer.with_batch(1).dims()
        assert rel_l2(got[img:img + 1], oracle_conv(x[img:img + 1], f, one)) <= TOL[mode]
    assert np.isfinite(got).all()


@pytest.mark.parametrize("mode", [b.MODE_TF32, b.MODE_BF16], ids=MODE_ID.get)
def test_conv_long_reduction_few_filters_sampled(mode):
    """Table I Conv4 (C = 64, 7x7, stride 2, K = 64: an 802 KB filter) at batch 16, where the library
    keeps one reduction slice of the filter per CTA and adds partial sums into the zeroed output.
    Checked at sampled output coordinates, the corners and the whole last image."""
    layer = wl.CONFIGS["table1_Conv4"].with_batch(16)
    dims = layer.dims()
    n, c, h, w, k, fh, fw, s = dims
    x, f = wl.make_input(layer), wl.make_filter(layer)
    got = gpu_conv(x, f, dims, mode)
    ho, wo = b.out_dims(dims)
    rng = np.random.default_rng(4321)
    idx = np.stack([rng.integers(0, n, 5000), rng.integers(0, k, 5000), rng.integers(0, ho, 5000),
                    rng.integers(0, wo, 5000)], axis=1).astype(np.int32)
    corners = np.array(list(itertools.product((0, n - 1), (0, k - 1), (0, ho - 1), (0, wo - 1))), dtype=np.int32)
    idx = np.concatenate([idx, corners])
    ref = oracle.conv_direct_points(x, f, oracle.Shape(*dims), idx)
    assert rel_l2(got[idx[:, 0], idx[:, 1], idx[:, 2], idx[:, 3]], ref) <= TOL[mode]
    one = layer.with_batch(1).dims()
    assert rel_l2(got[n - 1:n], oracle_conv(x[n - 1:n], f, one)) <= TOL[mode]
    assert np.isfinite(got).all()


@pytest.mark.parametrize("mode", [b.MODE_TF32, b.MODE_BF16, b.MODE_FP32], ids=MODE_ID.get)
@pytest.mark.parametrize("dims", [(19, 16, 30, 30, 32, 3, 3, 1), (3, 5, 17, 19, 7, 2, 3, 2), (1, 3, 32, 32, 16, 3, 3, 1)])
def test_conv_host_buffers(dims, mode):
    """im2win_conv_host: host buffers in and out (the batch is pipelined through the GPU in chunks)."""
    import torch
    n, c, h, w, k, fh, fw, s = dims
    x, f = _data(dims, 900)
    ho, wo = b.out_dims(dims)
    out = torch.full((n, k, ho, wo), float("nan"), dtype=torch.float32).pin_memory()
    for _ in range(2):
        b.conv_host(torch.from_numpy(x).pin_memory(), torch.from_numpy(f), dims, mode, out)
    assert rel_l2(out.numpy(), oracle_conv(x, f, dims)) <= TOL[mode]
    b.host_release()
