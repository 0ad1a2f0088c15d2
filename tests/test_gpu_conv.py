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
from gpu_helpers import CONV_CONFIGS, TOL, apply_config, ensure_built, gpu_conv, oracle_conv, rel_l2, reset_config

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
    # shapes the strip-matrix kernel takes (3x3, channels in multiples of 16 / 32): odd widths, filter counts
    # that are no multiple of 16, two filter tiles, stride 2 with odd and even widths, images smaller than a
    # tile and of a single output, several tiles per image
    (2, 16, 11, 13, 24, 3, 3, 1), (3, 32, 9, 10, 40, 3, 3, 2), (1, 64, 17, 19, 300, 3, 3, 1), (2, 32, 20, 33, 17, 3, 3, 2),
    (2, 64, 5, 5, 16, 3, 3, 1), (3, 32, 3, 3, 8, 3, 3, 1), (1, 32, 40, 37, 48, 3, 3, 1), (1, 32, 45, 44, 130, 3, 3, 2),
    # shapes for the window-offset kernel (stride 1, 3x3 and 5x5): a 5x5 filter, source ranges of several TMA
    # boxes, four 128-row blocks per tile with a ragged last tile
    (1, 32, 14, 15, 24, 5, 5, 1), (2, 64, 30, 28, 64, 3, 3, 1), (1, 32, 70, 66, 32, 3, 3, 1),
    # two filter tiles of 144: two blocks per tile leave one accumulator buffer, so the interleaver warps help
    # the epilogue (with two issuing threads they too must zero the columns they read)
    (2, 64, 20, 30, 288, 3, 3, 1),
    # pointwise and factorised filters (1x1; 1x3 / 3x1; 1x7 / 7x1): families of the persistent kernel; channel
    # counts of 32 (the pointwise groups), 16 and 8 (TF32 1x7), strides, two filter tiles, tiles that span images
    (3, 64, 9, 11, 40, 1, 1, 1), (2, 48, 14, 13, 300, 1, 1, 2), (2, 32, 12, 17, 24, 1, 3, 1), (2, 16, 17, 12, 33, 3, 1, 2),
    (1, 24, 9, 40, 20, 1, 7, 1), (2, 16, 30, 9, 130, 7, 1, 1), (4, 8, 6, 9, 16, 1, 7, 3),
    # patch / downsampling filters and 3x5 / 5x3 (also families of the persistent kernel)
    (2, 32, 18, 22, 40, 2, 2, 2), (2, 16, 36, 40, 24, 4, 4, 4), (2, 16, 13, 19, 300, 3, 5, 1), (1, 32, 21, 11, 17, 5, 3, 2),
]
RECT_FAMILIES = ((1, 1), (1, 3), (3, 1), (1, 7), (7, 1), (2, 2), (4, 4), (3, 5), (5, 3))
RECT_SHAPES = [d for d in SMALL if (d[5], d[6]) in RECT_FAMILIES and d[1] % 8 == 0]
STRIP_SHAPES = [d for d in SMALL if d[5] == 3 and d[6] == 3 and d[1] % 32 == 0 and d[7] in (1, 2)]
WINDOW_SHAPES = [d for d in SMALL if (d[5], d[6]) in ((3, 3), (5, 5)) and d[1] % 32 == 0 and d[7] == 1]


@pytest.fixture(scope="module", autouse=True)
def _built():
    ensure_built()


@pytest.fixture(params=list(CONV_CONFIGS), autouse=True)
def _kernel(request):
    """Every case runs once per kernel configuration: the product library's own choice ("auto"; the
    same with the smallest legal workspace, "minws"), and the test build with one switch set -- the
    strip-matrix kernel forced wherever it is implemented (one and two 128-row halves per tile), the
    window-offset kernel forced wherever it is implemented (its own tile height, one and two 128-row blocks), the
    strip-matrix kernel off (the persistent, filter-size-specialised kernel's own choice), that kernel
    with box staging off (per-image tiles, bulk copies), with per-image tiling off as well (tiles that
    span images), with three reduction slices forced, with the slice-resident filter mode forced, and
    the generic kernel forced."""
    apply_config(request.param)
    yield request.param
    reset_config()


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
@pytest.mark.parametrize("dims", STRIP_SHAPES)
def test_forced_strip_configurations_run_the_strip_kernel(dims, mode, _kernel):
    """The configurations that force the strip-matrix kernel must really run it on the shapes it
    implements (a silent fall-through to another kernel would leave it untested)."""
    if _kernel not in ("strip", "strip2", "pair", "pair2"):
        pytest.skip("only for the configurations that force the strip-matrix kernel")
    x, f = _data(dims, 800, ints=True)
    got = gpu_conv(x, f, dims, mode)
    if dims[7] == 1 or _kernel in ("strip", "pair"):  # (two halves per tile and stride 2 together exceed shared memory)
        assert b.last_kernel() == b.KERNEL_STRIP
    assert np.array_equal(got.astype(np.float64), oracle_conv(x, f, dims))


@pytest.mark.parametrize("src_kind", [b.SRC_NCHW, b.SRC_NCHW_FUSED], ids=["im2win", "fused"])
@pytest.mark.parametrize("mode", [b.MODE_TF32, b.MODE_BF16], ids=MODE_ID.get)
@pytest.mark.parametrize("dims", WINDOW_SHAPES)
def test_forced_window_configurations_run_the_window_kernel(dims, mode, src_kind, _kernel):
    """The same for the window-offset kernel, from the im2win tensor and fused."""
    if _kernel not in ("window", "window1", "window2", "wtwo", "wstream", "wpair", "wpair2"):
        pytest.skip("only for the configurations that force the window-offset kernel")
    x, f = _data(dims, 810, ints=True)
    got = gpu_conv(x, f, dims, mode, src_kind=src_kind)
    tiles = -(-dims[4] // 256)
    nt = -(-(-(-dims[4] // tiles)) // 16) * 16
    if not (_kernel.startswith("wpair") and nt % 32):  # (a pair splits the filter tile into two halves of whole 16-row groups)
        assert b.last_kernel() == b.KERNEL_WINDOW
    assert np.array_equal(got.astype(np.float64), oracle_conv(x, f, dims))


@pytest.mark.parametrize("src_kind", [b.SRC_NCHW, b.SRC_NCHW_FUSED], ids=["im2win", "fused"])
@pytest.mark.parametrize("mode", [b.MODE_TF32, b.MODE_BF16], ids=MODE_ID.get)
@pytest.mark.parametrize("dims", RECT_SHAPES)
def test_pointwise_and_factorised_filters_run_the_persistent_kernel(dims, mode, src_kind, _kernel):
    """1x1, 1x3 / 3x1, 1x7 / 7x1, 2x2, 4x4 and 3x5 / 5x3 filters are families of the persistent kernel, not cases
    of the generic one: the configurations that leave the choice to the library must run it (channel counts
    that are multiples of 16; in TF32 mode with seven or more taps: of 8)."""
    if _kernel not in ("nostrip", "nobox", "nopim", "split3", "bslice"):
        pytest.skip("only for the test-build configurations that leave the persistent kernel its own choice")
    x, f = _data(dims, 820, ints=True)
    got = gpu_conv(x, f, dims, mode, src_kind=src_kind)
    c, taps = dims[1], dims[5] * dims[6]
    if c % 16 == 0 or (mode == b.MODE_TF32 and taps >= 7):
        assert b.last_kernel() == b.KERNEL_PERSISTENT
    assert np.array_equal(got.astype(np.float64), oracle_conv(x, f, dims))


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


# Inputs and oracle results of the full-size cases, computed once per module (every case runs in
# several kernel configurations, and the oracle takes seconds per layer at batch 128).
_CACHE: dict = {}


def _cached(key, make):
    if key not in _CACHE:
        _CACHE[key] = make()
    return _CACHE[key]


def _layer_ints(layer):
    n, c, h, w, k, fh, fw, s = layer.dims()
    x = wl.small_ints(9000 + layer.seed, n * c * h * w).reshape(n, c, h, w)
    f = wl.small_ints(9500 + layer.seed, k * c * fh * fw, -2, 2).reshape(k, c, fh, fw)
    return x, f


def _exact_f32(ref64):
    """The oracle's fp64 result as fp32, after checking that the conversion loses nothing."""
    assert np.abs(ref64).max() < 2 ** 24 and np.array_equal(ref64, np.rint(ref64))
    return ref64.astype(np.float32)


FULL = ["resnet3x3", "stem7x7", "deep3x3", "down3x3"]


@pytest.mark.parametrize("mode", [b.MODE_TF32, b.MODE_BF16], ids=MODE_ID.get)
@pytest.mark.parametrize("src", ["nchw", "fused"])
@pytest.mark.parametrize("name", FULL)
def test_conv_full_batch_small_integers_whole_tensor_bit_exact(name, src, mode, _kernel):
    """Batch 128, the launch configuration the benchmark times (ring phases wrapping over ~170 tiles
    per CTA, the look-ahead of the next tile, the last partial wave): on small-integer data every one
    of the 6 to 103 million outputs must equal the oracle's Eq. (1) exactly."""
    if src == "fused" and _kernel not in ("auto", "strip", "window", "nostrip"):
        pytest.skip("the fused source kind is covered in the library's own, the strip-matrix, the window-offset and the persistent configuration")
    layer = wl.CONFIGS[name]
    dims = layer.dims()
    x, f = _cached(("ints", name), lambda: _layer_ints(layer))
    ref = _cached(("ints_ref", name), lambda: _exact_f32(oracle_conv(x, f, dims)))
    got = gpu_conv(x, f, dims, mode, src_kind=b.SRC_NCHW_FUSED if src == "fused" else b.SRC_NCHW)
    assert np.array_equal(got, ref)


@pytest.mark.parametrize("mode", [b.MODE_TF32, b.MODE_BF16], ids=MODE_ID.get)
@pytest.mark.parametrize("name", FULL)
def test_conv_full_batch_whole_tensor(name, mode):
    """Batch 128 on the benchmark's data: relative L2 over the WHOLE output against the oracle's Eq. (1),
    plus a bound on the largest single error (a wrong accumulator column in one tile of one image would
    move the norm by nothing, but is off by the size of an output, hundreds of times this bound)."""
    layer = wl.CONFIGS[name]
    dims = layer.dims()
    x, f = _cached(("real", name), lambda: (wl.make_input(layer), wl.make_filter(layer)))
    ref = _cached(("real_ref", name), lambda: oracle_conv(x, f, dims))
    got = gpu_conv(x, f, dims, mode)
    assert np.isfinite(got).all()
    assert rel_l2(got, ref) <= TOL[mode]
    rms = float(np.sqrt(np.mean(ref * ref)))
    assert float(np.abs(got - ref).max()) <= 8.0 * TOL[mode] * rms


@pytest.mark.parametrize("mode", [b.MODE_TF32, b.MODE_BF16], ids=MODE_ID.get)
@pytest.mark.parametrize("batch", [32, 128])
@pytest.mark.parametrize("layer", wl.SWEEP, ids=lambda l: l.name)
def test_conv_sweep_layers_batch_32_and_128(layer, batch, mode, _kernel):
    """The twelve-layer sweep at the batch sizes the benchmark times, with the library's own choice of
    path at each (reduction slices at 32, streamed filters and multi-wave persistent loops at 128): Eq. (1)
    at 20 000 sampled coordinates and every corner, and the whole first and last image."""
    if _kernel not in ("auto", "minws", "strip", "window", "nostrip"):
        pytest.skip("forced persistent-kernel variants are covered at small sizes")
    layer = layer.with_batch(batch)
    dims = layer.dims()
    n, c, h, w, k, fh, fw, s = dims
    ho, wo = b.out_dims(dims)

    def make():
        x, f = wl.make_input(layer), wl.make_filter(layer)
        rng = np.random.default_rng(77 + batch)
        idx = np.stack([rng.integers(0, n, 20000), rng.integers(0, k, 20000), rng.integers(0, ho, 20000),
                        rng.integers(0, wo, 20000)], axis=1).astype(np.int32)
        corners = np.array(list(itertools.product((0, n - 1), (0, k - 1), (0, ho - 1), (0, wo - 1))), dtype=np.int32)
        idx = np.concatenate([idx, corners])
        pts = oracle.conv_direct_points(x, f, oracle.Shape(*dims), idx)
        one = layer.with_batch(1).dims()
        ends = {img: oracle_conv(x[img:img + 1], f, one) for img in (0, n - 1)}
        return x, f, idx, pts, ends

    x, f, idx, pts, ends = _cached(("sweep", layer.name, batch), make)
    got = gpu_conv(x, f, dims, mode)
    assert np.isfinite(got).all()
    sample = got[idx[:, 0], idx[:, 1], idx[:, 2], idx[:, 3]]
    assert rel_l2(sample, pts) <= TOL[mode]
    rms = float(np.sqrt(np.mean(pts * pts)))
    assert float(np.abs(sample - pts).max()) <= 8.0 * TOL[mode] * rms
    for img, ref in ends.items():
        assert rel_l2(got[img:img + 1], ref) <= TOL[mode]


@pytest.mark.parametrize("mode", [b.MODE_TF32, b.MODE_BF16], ids=MODE_ID.get)
@pytest.mark.parametrize("layer", [l for l in wl.TABLE_I_LAYERS if l.name != "table1_Conv4"], ids=lambda l: l.name)
def test_conv_table1_layers_batch128(layer, mode, _kernel):
    """The paper's own workload: Table I's unpadded layers at batch 128 (Conv4, whose tensors take
    gigabytes, is covered at batch 16 below).  Eq. (1) at 20 000 sampled coordinates and every corner,
    the whole first and last image, and no element that is not finite."""
    if _kernel not in ("auto", "minws", "strip", "pair2", "window", "nostrip"):
        pytest.skip("forced persistent-kernel variants are covered at small sizes")
    dims = layer.dims()
    n, c, h, w, k, fh, fw, s = dims
    ho, wo = b.out_dims(dims)

    def make():
        x, f = wl.make_input(layer), wl.make_filter(layer)
        rng = np.random.default_rng(99)
        idx = np.stack([rng.integers(0, n, 20000), rng.integers(0, k, 20000), rng.integers(0, ho, 20000),
                        rng.integers(0, wo, 20000)], axis=1).astype(np.int32)
        corners = np.array(list(itertools.product((0, n - 1), (0, k - 1), (0, ho - 1), (0, wo - 1))), dtype=np.int32)
        idx = np.concatenate([idx, corners])
        pts = oracle.conv_direct_points(x, f, oracle.Shape(*dims), idx)
        one = layer.with_batch(1).dims()
        ends = {img: oracle_conv(x[img:img + 1], f, one) for img in (0, n - 1)}
        return x, f, idx, pts, ends

    x, f, idx, pts, ends = _cached(("table1", layer.name), make)
    got = gpu_conv(x, f, dims, mode)
    assert np.isfinite(got).all()
    sample = got[idx[:, 0], idx[:, 1], idx[:, 2], idx[:, 3]]
    assert rel_l2(sample, pts) <= TOL[mode]
    rms = float(np.sqrt(np.mean(pts * pts)))
    assert float(np.abs(sample - pts).max()) <= 8.0 * TOL[mode] * rms
    for img, ref in ends.items():
        assert rel_l2(got[img:img + 1], ref) <= TOL[mode]


@pytest.mark.parametrize("mode", [b.MODE_TF32, b.MODE_BF16], ids=MODE_ID.get)
@pytest.mark.parametrize("layer", wl.SWEEP, ids=lambda l: l.name)
def test_conv_sweep_layers_batch32_small_integers_bit_exact(layer, mode, _kernel):
    if _kernel not in ("auto", "minws", "strip", "window", "wtwo", "wpair", "wpair2", "nostrip"):
        pytest.skip("forced persistent-kernel variants are covered at small sizes")
    layer = layer.with_batch(32)
    dims = layer.dims()
    x, f = _cached(("ints", layer.name, 32), lambda: _layer_ints(layer))
    ref = _cached(("ints_ref", layer.name, 32), lambda: _exact_f32(oracle_conv(x, f, dims)))
    assert np.array_equal(gpu_conv(x, f, dims, mode), ref)


@pytest.mark.parametrize("mode", [b.MODE_TF32, b.MODE_BF16], ids=MODE_ID.get)
@pytest.mark.parametrize("name", ["resnet3x3", "deep3x3"])
def test_conv_fifty_repeats_are_bit_identical_on_exact_data(name, mode, _kernel):
    """Several threads may issue the MMAs of one tile onto the same accumulator; a lost update would
    show as a run that differs.  Fifty runs at batch 128 on small-integer data, compared on the device."""
    import torch
    if _kernel not in ("auto", "nostrip", "split3"):
        pytest.skip("one configuration per kernel family")
    layer = wl.CONFIGS[name]
    dims = layer.dims()
    x, f = _cached(("ints", name), lambda: _layer_ints(layer))
    ho, wo = b.out_dims(dims)
    xd, fd = torch.from_numpy(x).cuda(), torch.from_numpy(f).cuda()
    ws = torch.empty(b.conv_workspace_bytes(dims, b.SRC_NCHW, mode) // 4, dtype=torch.float32, device="cuda")
    outs = [torch.empty((layer.N, layer.K, ho, wo), dtype=torch.float32, device="cuda") for _ in range(2)]
    b.conv(xd, b.SRC_NCHW, fd, dims, mode, outs[0], ws)
    for _ in range(50):
        outs[1].fill_(float("nan"))
        b.conv(ws, b.SRC_IM2WIN, fd, dims, mode, outs[1], ws[b.workspace_bytes(dims) // 4:] if ws.numel() > b.workspace_bytes(dims) // 4 + 64 else None)
        assert torch.equal(outs[0], outs[1])
    assert b.last_device_status() == 0
    ref = _cached(("ints_ref", name), lambda: _exact_f32(oracle_conv(x, f, dims)))
    assert np.array_equal(outs[0].cpu().numpy(), ref)


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
