"""im2win_conv_nhwc: the convolution's fp32 result written channels-last, against the oracle's Eq. (1)
transposed, through every kernel configuration (each kernel has the layout as an epilogue option)."""
import numpy as np
import pytest

import oracle
from paper_2306_14320_b200 import binding as b
from paper_2306_14320_b200 import workloads as wl
from gpu_helpers import CONV_CONFIGS, Guarded, TOL, apply_config, conv_workspace_floats, ensure_built, oracle_conv, rel_l2, reset_config

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

MODES = [b.MODE_TF32, b.MODE_BF16, b.MODE_FP32]
MODE_ID = {b.MODE_FP32: "fp32", b.MODE_TF32: "tf32", b.MODE_BF16: "bf16"}
# odd filter counts (scalar stores), K > 256 (two filter tiles), tiles that span images, strip / window shapes,
# 5x5, 7x7 stride 2, a rectangular filter (generic kernel)
SHAPES = [
    (2, 3, 9, 11, 5, 3, 3, 1), (1, 9, 40, 41, 300, 3, 3, 2), (5, 7, 9, 9, 17, 3, 3, 1), (2, 3, 37, 35, 24, 7, 7, 2),
    (1, 24, 20, 21, 300, 3, 3, 1), (2, 16, 11, 13, 24, 3, 3, 1), (1, 64, 17, 19, 300, 3, 3, 1), (2, 64, 30, 28, 64, 3, 3, 1),
    (1, 32, 14, 15, 24, 5, 5, 1), (1, 32, 45, 44, 130, 3, 3, 2), (1, 4, 12, 14, 6, 2, 3, 1), (1, 32, 70, 66, 32, 3, 3, 1),
]
SRC_ID = {b.SRC_NCHW: "im2win", b.SRC_NCHW_FUSED: "fused"}


@pytest.fixture(scope="module", autouse=True)
def _built():
    ensure_built()


@pytest.fixture(params=list(CONV_CONFIGS), autouse=True)
def _kernel(request):
    apply_config(request.param)
    yield request.param
    reset_config()


def gpu_conv_nhwc(x, f, dims, mode, src_kind=b.SRC_NCHW):
    n, c, h, w, k, fh, fw, s = dims
    ho, wo = b.out_dims(dims)
    xd = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).cuda()
    fd = torch.from_numpy(np.ascontiguousarray(f, dtype=np.float32)).cuda()
    out = Guarded(n * k * ho * wo)
    ws = Guarded(conv_workspace_floats(dims, src_kind, mode))
    b.conv_nhwc(xd, src_kind, fd, dims, mode, out.view, ws.view, ws.n * 4)
    assert b.last_device_status() == 0
    ws.check()
    return out.check().reshape(n, ho, wo, k)


def _ints(dims, seed):
    n, c, h, w, k, fh, fw, s = dims
    x = wl.small_ints(seed, n * c * h * w).reshape(n, c, h, w)
    f = wl.small_ints(seed + 1, k * c * fh * fw, -2, 2).reshape(k, c, fh, fw)
    return x, f


@pytest.mark.parametrize("src_kind", [b.SRC_NCHW, b.SRC_NCHW_FUSED], ids=SRC_ID.get)
@pytest.mark.parametrize("mode", MODES, ids=MODE_ID.get)
@pytest.mark.parametrize("dims", SHAPES)
def test_nhwc_small_integers_bit_exact(dims, mode, src_kind):
    x, f = _ints(dims, 900)
    got = gpu_conv_nhwc(x, f, dims, mode, src_kind)
    ref = np.transpose(oracle_conv(x, f, dims), (0, 2, 3, 1))
    assert np.array_equal(got.astype(np.float64), ref)


@pytest.mark.parametrize("mode", MODES, ids=MODE_ID.get)
@pytest.mark.parametrize("dims", SHAPES[:6])
def test_nhwc_real_data(dims, mode):
    n, c, h, w, k, fh, fw, s = dims
    x = wl.normal01(910, n * c * h * w).reshape(n, c, h, w)
    f = (wl.normal01(911, k * c * fh * fw) * np.float32(np.sqrt(2.0 / (c * fh * fw)))).reshape(k, c, fh, fw)
    got = gpu_conv_nhwc(x, f, dims, mode)
    assert rel_l2(got, np.transpose(oracle_conv(x, f, dims), (0, 2, 3, 1))) <= TOL[mode]


@pytest.mark.parametrize("mode", [b.MODE_TF32, b.MODE_BF16], ids=MODE_ID.get)
@pytest.mark.parametrize("name,batch", [("resnet3x3", 128), ("deep3x3", 128), ("sweep_L10", 32), ("sweep_L2", 32), ("stem7x7", 8)])
def test_nhwc_layers_small_integers_whole_tensor_bit_exact(name, batch, mode, _kernel):
    if _kernel not in ("auto", "strip", "pair2", "window", "wpair2", "nostrip"):
        pytest.skip("one configuration per kernel family at full size")
    layer = wl.CONFIGS[name].with_batch(batch)
    dims = layer.dims()
    x, f = _ints(dims, 920)
    got = gpu_conv_nhwc(x, f, dims, mode)
    ref = np.transpose(oracle_conv(x, f, dims), (0, 2, 3, 1)).astype(np.float32)
    assert np.array_equal(got, ref)


def test_nhwc_rejects_nothing_new_and_checks_arguments():
    dims = (1, 3, 8, 8, 4, 3, 3, 1)
    ho, wo = b.out_dims(dims)
    x = torch.zeros(3 * 64, device="cuda")
    f = torch.zeros(4 * 27, device="cuda")
    out = torch.zeros(4 * ho * wo, device="cuda")
    with pytest.raises(b.Im2winError) as exc:  # the transform needs a workspace, as in im2win_conv
        b.conv_nhwc(x, b.SRC_NCHW, f, dims, b.MODE_TF32, out, None)
    assert exc.value.code == b.EWORKSPACE
