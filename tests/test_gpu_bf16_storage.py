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
from gpu_helpers import GUARD, TOL, Guarded, ensure_built, oracle_conv, rel_l2

pytestmark = pytest.mark.gpu

SMALL = [
    (1, 1, 4, 4, 1, 2, 2, 1), (2, 3, 7, 9, 4, 3, 3, 1), (1, 2, 9, 8, 3, 2, 3, 1), (2, 2, 8, 11, 2, 3, 2, 2),
    (1, 3, 13, 12, 2, 4, 2, 3), (3, 5, 33, 37, 2, 3, 3, 1), (2, 3, 64, 64, 2, 5, 5, 2),
    (1, 2, 130, 1031, 1, 7, 7, 2), (1, 1, 30, 5000, 1, 11, 3, 4), (1, 1, 1, 1, 1, 1, 1, 1),
    (3, 50, 11, 11, 2, 2, 2, 4), (2, 700, 9, 9, 2, 3, 3, 1),
]
# layers whose images are large enough for per-image tiling (the variant's stated limit)
LAYERS = [("resnet3x3", 3), ("stem7x7", 1), ("sweep_L1", 1), ("sweep_L6", 2), ("sweep_L8", 1), ("sweep_L9", 2)]


@pytest.fixture(scope="module", autouse=True)
def _built():
    ensure_built()


@pytest.fixture(params=["auto", "gather"], autouse=True)
def _kernel(request, monkeypatch):
    """Every case runs with the library's own choice of transform kernel (the TMA tile kernel where it
    applies) and with the staged-gather kernel forced."""
    monkeypatch.setenv("IM2WIN_TRANSFORM_GATHER", "1" if request.param == "gather" else "0")


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
    b.conv(ihat16.view, b.SRC_IM2WIN_BF16, fd, dims, b.MODE_BF16, out.view)
    assert b.last_device_status() == 0
    return out.check().reshape(n, k, ho, wo)


@pytest.mark.parametrize("dims", SMALL)
def test_transform_bf16_bit_exact_small(dims):
    n, c, h, w = dims[:4]
    x = wl.normal01(300 + h * w, n * c * h * w).reshape(n, c, h, w)
    x.reshape(-1)[::97] = np.float32(-0.0)
    ref = bf16_rne_bits(oracle.im2win(x, oracle.Shape(*dims)))
    assert np.array_equal(gpu_transform_bf16(x, dims).check(), ref)


@pytest.mark.parametrize("name,batch", LAYERS + [("deep3x3", 3), ("down3x3", 2)])
def test_transform_bf16_bit_exact_layer_shapes(name, batch):
    layer = wl.CONFIGS[name].with_batch(batch)
    x = wl.make_input(layer)
    ref = bf16_rne_bits(oracle.im2win(x, oracle.Shape(*layer.dims())))
    assert np.array_equal(gpu_transform_bf16(x, layer.dims()).check(), ref)


@pytest.mark.parametrize("staging", ["box", "bulk"])
@pytest.mark.parametrize("name,batch", LAYERS)
def test_conv_from_bf16_im2win_tensor(name, batch, staging, monkeypatch):
    monkeypatch.setenv("IM2WIN_NO_BOX", "1" if staging == "bulk" else "0")
    layer = wl.CONFIGS[name].with_batch(batch)
    dims = layer.dims()
    x, f = wl.make_input(layer), wl.make_filter(layer)
    got = gpu_conv_from_bf16(gpu_transform_bf16(x, dims), f, dims)
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
    small = wl.CONFIGS["deep3x3"].with_batch(1)  # images too small for per-image tiling: stated limit
    sd = small.dims()
    s16 = gpu_transform_bf16(wl.make_input(small), sd)
    sf = torch.from_numpy(wl.make_filter(small)).cuda()
    sho, swo = b.out_dims(sd)
    sout = torch.empty(small.N * small.K * sho * swo, device="cuda")
    with pytest.raises(b.Im2winError) as e:
        b.conv(s16.view, b.SRC_IM2WIN_BF16, sf, sd, b.MODE_BF16, sout)
    assert e.value.code == b.EUNSUPPORTED
