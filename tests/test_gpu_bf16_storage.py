"""GPU parity, bf16 storage variant of the im2win tensor (a storage mode of this build; the paper stores
fp32 only): `im2win_transform_bf16` must equal the oracle's Algorithm 1 rounded to bf16 (nearest even)
bit for bit, and a BF16-mode convolution that reads that tensor must meet the BF16 tolerance against
the oracle's Eq. (1) -- its MMA operands are the same bf16 values as from an fp32 im2win tensor."""
import numpy as np
import pytest
import torch

import oracle
from paper_2306_14320_b200 import binding as b
from paper_2306_14320_b200 import workloads as wl
from gpu_helpers import GUARD, TOL, Guarded, apply_config, conv_workspace_floats, ensure_built, oracle_conv, rel_l2, reset_config

pytestmark = pytest.mark.gpu

SMALL = [
    (1, 1, 4, 4, 1, 2, 2, 1), (2, 3, 7, 9, 4, 3, 3, 1), (1, 2, 9, 8, 3, 2, 3, 1), (2, 2, 8, 11, 2, 3, 2, 2),
    (1, 3, 13, 12, 2, 4, 2, 3), (3, 5, 33, 37, 2, 3, 3, 1), (2, 3, 64, 64, 2, 5, 5, 2),
    (1, 2, 130, 1031, 1, 7, 7, 2), (1, 1, 30, 5000, 1, 11, 3, 4), (1, 1, 1, 1, 1, 1, 1, 1),
    (3, 50, 11, 11, 2, 2, 2, 4), (2, 700, 9, 9, 2, 3, 3, 1),
]
# every named layer and every layer of the sweep: the persistent kernel reads a bf16 im2win tensor where
# its tiles are cut per image, the strip-matrix kernel takes the 3x3 layers with small images
LAYERS = [("resnet3x3", 3), ("stem7x7", 1), ("deep3x3", 3), ("down3x3", 2)] + [(l.name, 2) for l in wl.SWEEP]


@pytest.fixture(scope="module", autouse=True)
def _built():
    ensure_built()


@pytest.fixture(params=["auto", "gather"], autouse=True)
def _kernel(request):
    """Every case runs with the product library's own choice of transform kernel (the TMA tile kernel
    where it applies) and with the staged-gather kernel forced (a switch of the test build)."""
    apply_config("gather" if request.param == "gather" else "auto", **({"transform_gather": 1} if request.param == "gather" else {}))
    yield request.param
    reset_config()


def bf16_rne_bits(a: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 bit patterns, round to nearest even (finite inputs), in numpy."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32).astype(np.uint64)
    return ((u + 0x7FFF + ((u >> 16) & 1)) >> 16).astype(np.uint16).ravel()


class Guarded16:
    """n 16-bit words on the device between sentinel guard bands."""

    def __init__(self, n: int):
        self.n = n
        self.full = torch.full((n + 2 * GUARD,), 0x7BAD, dtype=torch.int16, device="cuda")
        self.view = self.full[GUARD:GUARD + n]
        assert self.view.data_ptr() % 16 == 0

    def check(self) -> np.ndarray:
        host = self.full.cpu().numpy()
        assert np.all(host[:GUARD] == 0x7BAD), "write before the buffer"
        assert np.all(host[GUARD + self.n:] == 0x7BAD), "write past the buffer"
        return host[GUARD:GUARD + self.n].view(np.uint16)


def gpu_transform_bf16(x: np.ndarray, dims) -> Guarded16:
    xd = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).cuda()
    assert b.workspace_bytes_bf16(dims) * 2 == b.workspace_bytes(dims)
    out = Guarded16(b.workspace_bytes_bf16(dims) // 2)
    b.transform_bf16(xd, dims, out.view)
    assert b.last_device_status() == 0
    return out


def gpu_conv_from_bf16(ihat16: Guarded16, f: np.ndarray, dims) -> np.ndarray:
    n, c, h, w, k, fh, fw, s = dims
    ho, wo = b.out_dims(dims)
    fd = torch.from_numpy(np.ascontiguousarray(f, dtype=np.float32)).cuda()
    out = Guarded(n * k * ho * wo)
    ws = Guarded(max(64, b.conv_workspace_bytes(dims, b.SRC_IM2WIN_BF16, b.MODE_BF16) // 4))  # scratch for a filter copy
    b.conv(ihat16.view, b.SRC_IM2WIN_BF16, fd, dims, b.MODE_BF16, out.view, ws.view, ws.n * 4)
    assert b.last_device_status() == 0
    ws.check()
    return out.check().reshape(n, k, ho, wo)


@pytest.mark.parametrize("dims", SMALL)
def test_transform_bf16_bit_exact_small(dims):
    n, c, h, w = dims[:4]
    x = wl.normal01(300 + h * w, n * c * h * w).reshape(n, c, h, w)
    x.reshape(-1)[::97] = np.float32(-0.0)
    ref = bf16_rne_bits(oracle.im2win(x, oracle.Shape(*dims)))
    assert np.array_equal(gpu_transform_bf16(x, dims).check(), ref)


@pytest.mark.parametrize("name,batch", LAYERS)
def test_transform_bf16_bit_exact_layer_shapes(name, batch):
    layer = wl.CONFIGS[name].with_batch(batch)
    x = wl.make_input(layer)
    ref = bf16_rne_bits(oracle.im2win(x, oracle.Shape(*layer.dims())))
    assert np.array_equal(gpu_transform_bf16(x, layer.dims()).check(), ref)


@pytest.mark.parametrize("staging", ["auto", "box", "bulk"])
@pytest.mark.parametrize("name,batch", LAYERS)
def test_conv_from_bf16_im2win_tensor(name, batch, staging, _kernel):
    """staging: the library's own choice of kernel; the persistent kernel with 2-D TMA boxes; the same
    with bulk copies."""
    if staging != "auto":
        apply_config(staging, no_strip=1, no_window=1, no_box=1 if staging == "bulk" else 0, transform_gather=1 if _kernel == "gather" else 0)
    layer = wl.CONFIGS[name].with_batch(batch)
    dims = layer.dims()
    x, f = wl.make_input(layer), wl.make_filter(layer)
    try:
        got = gpu_conv_from_bf16(gpu_transform_bf16(x, dims), f, dims)
    except b.Im2winError as exc:
        if staging != "auto" and exc.code == b.EUNSUPPORTED:
            pytest.skip("with the strip-matrix kernel switched off, no kernel reads a bf16 tensor of this layer")
        raise
    assert rel_l2(got, oracle_conv(x, f, dims)) <= TOL[b.MODE_BF16]
    # the same bf16 operands as the BF16 mode reading an fp32 im2win tensor: equal up to the order
    # of the fp32 additions
    from gpu_helpers import gpu_conv
    via_fp32 = gpu_conv(x, f, dims, b.MODE_BF16)
    np.testing.assert_allclose(got, via_fp32, rtol=1e-4, atol=1e-4)


def test_conv_from_bf16_small_integers_bit_exact():
    """Small integers are exact in bf16 and their sums exact in fp32: the result must equal Eq. (1)."""
    layer = wl.CONFIGS["resnet3x3"].with_batch(2)
    dims = layer.dims()
    n, c, h, w, k, fh, fw, s = dims
    x = wl.small_ints(11, n * c * h * w).reshape(n, c, h, w)
    f = wl.small_ints(12, k * c * fh * fw, -2, 2).reshape(k, c, fh, fw)
    got = gpu_conv_from_bf16(gpu_transform_bf16(x, dims), f, dims)
    assert np.array_equal(got.astype(np.float64), oracle_conv(x, f, dims))


def test_bf16_source_argument_checks():
    layer = wl.CONFIGS["resnet3x3"].with_batch(1)
    dims = layer.dims()
    ihat16 = gpu_transform_bf16(wl.make_input(layer), dims)
    fd = torch.from_numpy(wl.make_filter(layer)).cuda()
    ho, wo = b.out_dims(dims)
    out = torch.empty(layer.N * layer.K * ho * wo, device="cuda")
    with pytest.raises(b.Im2winError) as e:  # a bf16 tensor cannot feed the TF32 mode
        b.conv(ihat16.view, b.SRC_IM2WIN_BF16, fd, dims, b.MODE_TF32, out)
    assert e.value.code == b.EINVAL
    small = wl.Layer("odd", 1, 24, 12, 12, 16, 3, 3, 1)  # small images and a channel count no 16-bit kernel takes
    sd = small.dims()
    s16 = gpu_transform_bf16(wl.make_input(small), sd)
    sf = torch.from_numpy(wl.make_filter(small)).cuda()
    sho, swo = b.out_dims(sd)
    sout = torch.empty(small.N * small.K * sho * swo, device="cuda")
    with pytest.raises(b.Im2winError) as e:
        b.conv(s16.view, b.SRC_IM2WIN_BF16, sf, sd, b.MODE_BF16, sout)
    assert e.value.code == b.EUNSUPPORTED


# ------------------------------------------------------------------ bf16 OUTPUT (im2win_conv_bf16out)

def _bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def gpu_conv_bf16out(x: np.ndarray, f: np.ndarray, dims, mode: int, src_kind: int) -> np.ndarray:
    n, c, h, w, k, fh, fw, s = dims
    ho, wo = b.out_dims(dims)
    xd = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).cuda()
    fd = torch.from_numpy(np.ascontiguousarray(f, dtype=np.float32)).cuda()
    out = Guarded16(n * k * ho * wo)
    ws = Guarded(conv_workspace_floats(dims, src_kind, mode))
    b.conv_bf16out(xd, src_kind, fd, dims, mode, out.view, ws.view, ws.n * 4)
    assert b.last_device_status() == 0
    ws.check()
    return out.check().reshape(n, k, ho, wo)


# tolerance: the mode's own, plus the rounding of the result to bf16 (relative 2^-9 at most)
TOL_OUT = {b.MODE_TF32: 5e-3 + 2.0 ** -9, b.MODE_BF16: 2e-2 + 2.0 ** -9}


@pytest.mark.parametrize("mode", [b.MODE_TF32, b.MODE_BF16], ids=["tf32", "bf16"])
@pytest.mark.parametrize("src_kind", [b.SRC_NCHW, b.SRC_NCHW_FUSED], ids=["nchw", "fused"])
@pytest.mark.parametrize("name,batch", [("tiny", 1), ("resnet3x3", 3), ("stem7x7", 1), ("deep3x3", 3), ("down3x3", 2),
                                        ("sweep_L1", 1), ("sweep_L2", 1), ("sweep_L12", 2)])
def test_conv_bf16_output(name, batch, src_kind, mode):
    """Odd and even images sizes (tiny: 30x30 outputs; sweep_L1: 55x55, odd; sweep_L12: 7x7 with tiles
    that span images), resident and streamed filters."""
    layer = wl.CONFIGS[name].with_batch(batch)
    dims = layer.dims()
    x, f = wl.make_input(layer), wl.make_filter(layer)
    got = _bf16_bits_to_f64(gpu_conv_bf16out(x, f, dims, mode, src_kind))
    assert rel_l2(got, oracle_conv(x, f, dims)) <= TOL_OUT[mode]


@pytest.mark.parametrize("dims", [(2, 16, 30, 30, 32, 3, 3, 1), (3, 8, 21, 23, 40, 3, 3, 2), (2, 3, 37, 35, 24, 7, 7, 2)])
def test_conv_bf16_output_small_integers_bit_exact(dims):
    """Exact fp32 sums (small integers): the stored words must be the oracle's Eq. (1) rounded to bf16."""
    n, c, h, w, k, fh, fw, s = dims
    x = wl.small_ints(21, n * c * h * w).reshape(n, c, h, w)
    f = wl.small_ints(22, k * c * fh * fw, -2, 2).reshape(k, c, fh, fw)
    ref = oracle_conv(x, f, dims).astype(np.float32)
    for mode in (b.MODE_TF32, b.MODE_BF16):
        got = gpu_conv_bf16out(x, f, dims, mode, b.SRC_NCHW)
        assert np.array_equal(got.ravel(), bf16_rne_bits(ref))


def test_conv_bf16_output_argument_checks():
    layer = wl.CONFIGS["tiny"]
    dims = layer.dims()
    xd = torch.from_numpy(wl.make_input(layer)).cuda()
    fd = torch.from_numpy(wl.make_filter(layer)).cuda()
    ho, wo = b.out_dims(dims)
    out = torch.empty(layer.N * layer.K * ho * wo, dtype=torch.int16, device="cuda")
    ws = torch.empty(b.workspace_bytes(dims) // 4, device="cuda")
    with pytest.raises(b.Im2winError) as e:  # the fp32 check mode has no bf16 output
        b.conv_bf16out(xd, b.SRC_NCHW, fd, dims, b.MODE_FP32, out, ws)
    assert e.value.code == b.EINVAL
    odd = (1, 2, 9, 8, 3, 2, 3, 1)  # 2x3 filter: no specialised kernel, hence no bf16 epilogue
    n, c, h, w, k, fh, fw, s = odd
    oh, ow = b.out_dims(odd)
    with pytest.raises(b.Im2winError) as e:
        b.conv_bf16out(torch.zeros(n * c * h * w, device="cuda"), b.SRC_NCHW, torch.zeros(k * c * fh * fw, device="cuda"),
                       odd, b.MODE_TF32, torch.empty(n * k * oh * ow, dtype=torch.int16, device="cuda"),
                       torch.empty(b.workspace_bytes(odd) // 4, device="cuda"))
    assert e.value.code == b.EUNSUPPORTED
