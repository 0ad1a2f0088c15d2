"""Pins for the CPU oracle: every check here compares the oracle with something that is not the
oracle -- numbers the paper prints, closed forms, structural invariants, textbook special cases,
an independent library convolution, and brute force on tiny inputs."""
import itertools

import numpy as np
import pytest
import torch

import oracle
from oracle import Shape
from paper_2306_14320_b200 import workloads as wl
from conftest import golden_path


def _read_golden_kv(name):
    kv = {}
    with open(golden_path(name)) as fh:
        for line in fh:
            line = line.split("#")[0].strip()
            if line:
                k, *v = line.split()
                kv[k] = v
    return kv


def _rand(shape, seed):
    return wl.normal01(seed, int(np.prod(shape))).reshape(shape)


TINY_SHAPES = [
    # N, C, H, W, K, Fh, Fw, s  -- square, rectangular (Fh != Fw), strides up to 4, sizes that the
    # stride does not divide, Fh <= s and s > Fh included.
    (1, 1, 4, 4, 2, 2, 2, 1), (2, 3, 7, 9, 4, 3, 3, 1), (1, 2, 9, 8, 3, 2, 3, 1), (2, 2, 8, 11, 2, 3, 2, 2),
    (1, 3, 13, 12, 2, 4, 2, 3), (1, 1, 10, 10, 1, 1, 1, 1), (2, 2, 6, 6, 3, 2, 2, 2), (1, 2, 11, 7, 2, 2, 2, 3),
    (1, 1, 12, 13, 2, 1, 3, 4), (1, 2, 5, 5, 2, 5, 5, 1), (1, 3, 9, 9, 5, 3, 1, 2), (2, 1, 13, 13, 2, 4, 4, 4),
]


# ---------------------------------------------------------------- paper-printed numbers
def test_worked_example_counts_and_strips():
    g = _read_golden_kv("worked_example_4x4.txt")
    sh = Shape(1, 1, 4, 4, 1, 2, 2, 1)
    x = np.arange(16, dtype=np.float32).reshape(1, 1, 4, 4)
    xhat = oracle.im2win(x, sh)
    assert x.size == int(g["input_elements"][0])
    assert xhat.size == int(g["im2win_elements"][0])
    # the im2col count comes from the matrix the oracle really builds, not from a formula
    _, m_elems = oracle.conv_via_im2col(x, np.ones((1, 1, 2, 2), np.float32), sh)
    assert m_elems == int(g["im2col_elements"][0])
    assert xhat.shape == (1, 1, 3, 8)
    for m in range(3):
        assert xhat[0, 0, m].tolist() == [float(t) for t in g[f"strip{m}"]]
    # "1/3 less elements than the im2col matrix"
    assert (m_elems - xhat.size) * 3 == m_elems
    c = oracle.counts(sh)
    assert (c["input"], c["im2win"], c["im2col"]) == (16, 24, 36)


def test_table1_output_sizes_floor_division():
    rows = []
    with open(golden_path("table1_output_sizes.txt")) as fh:
        for line in fh:
            line = line.split("#")[0].split()
            if line:
                rows.append((line[0], *map(int, line[1:])))
    assert len(rows) == 12
    assert [r[1:6] for r in rows] == [tuple(t) for t in wl.TABLE_I]
    for name, c, h, k, f, s, ho_printed in rows:
        ho, wo = oracle.out_dims(Shape(128, c, h, h, k, f, f, s))
        assert (ho, wo) == (ho_printed, ho_printed), name
    # Conv4: (224-7)/2 = 108.5 -> the printed 109 needs floor
    assert oracle.out_dims(Shape(1, 64, 224, 224, 64, 7, 7, 2)) == (109, 109)


def test_table1_mean_size_ratio_2p93():
    g = _read_golden_kv("worked_example_4x4.txt")
    ratios = []
    for c, h, k, f, s in wl.TABLE_I:
        cnt = oracle.counts(Shape(128, c, h, h, k, f, f, s))
        ratios.append(cnt["im2col"] / cnt["im2win"])
    assert round(float(np.mean(ratios)), 2) == float(g["mean_im2col_over_im2win_table1"][0])


# ---------------------------------------------------------------- closed forms (Section III-A)
def _all_layers():
    out = [(l.name, Shape(*l.dims())) for l in wl.CONFIGS.values()]
    return out


@pytest.mark.parametrize("name,sh", _all_layers())
def test_closed_form_counts(name, sh):
    ho, wo = oracle.out_dims(sh)
    c = oracle.counts(sh)
    assert ho == (sh.H - sh.Fh) // sh.s + 1 and wo == (sh.W - sh.Fw) // sh.s + 1
    assert c["input"] == sh.N * sh.C * sh.H * sh.W
    assert c["im2win"] == sh.N * sh.C * sh.Fh * sh.W * ho
    assert c["im2col"] == sh.N * sh.C * sh.Fh * sh.Fw * ho * wo
    assert c["output"] == sh.N * sh.K * ho * wo
    # size independent of Wf
    for fw in (1, 2, sh.Fw + 1):
        if fw <= sh.W:
            assert oracle.counts(Shape(sh.N, sh.C, sh.H, sh.W, sh.K, sh.Fh, fw, sh.s))["im2win"] == c["im2win"]
    # the paper's delta = Hf*Ci*(Wi-Wf)*Ho*(Wf/s-1), valid when s divides Wi-Wf and Wf
    if sh.Fh == sh.Fw and (sh.W - sh.Fw) % sh.s == 0:
        delta = sh.Fh * sh.C * (sh.W - sh.Fw) * ho * (sh.Fw / sh.s - 1)
        assert (c["im2col"] - c["im2win"]) / sh.N == pytest.approx(delta, rel=1e-12)
    assert c["im2col"] >= c["im2win"] or sh.Fw < sh.s


def test_sizes_equal_input_when_filter_equals_stride():
    # Hf = Wf = s with exact division: im2win, im2col and the input all have the same size
    for (h, f) in [(8, 2), (9, 3), (16, 4)]:
        c = oracle.counts(Shape(2, 3, h, h, 4, f, f, f))
        assert c["im2win"] == c["im2col"] == c["input"]


def test_counts_match_materialised_tensors():
    for dims in TINY_SHAPES:
        sh = Shape(*dims)
        x = _rand((sh.N, sh.C, sh.H, sh.W), 5)
        f = _rand((sh.K, sh.C, sh.Fh, sh.Fw), 6)
        c = oracle.counts(sh)
        assert oracle.im2win(x, sh).size == c["im2win"]
        assert oracle.conv_via_im2col(x, f, sh)[1] * sh.N == c["im2col"]


# ---------------------------------------------------------------- transform: invariants and brute force
@pytest.mark.parametrize("dims", TINY_SHAPES)
def test_im2win_bruteforce_gather(dims):
    """Every element of the im2win tensor is looked up independently from its defining index map
    (numpy fancy indexing, no loops shared with the oracle)."""
    sh = Shape(*dims)
    x = _rand((sh.N, sh.C, sh.H, sh.W), 11)
    xhat = oracle.im2win(x, sh)
    ho, _ = oracle.out_dims(sh)
    assert xhat.shape == (sh.N, sh.C, ho, sh.W * sh.Fh)
    m, e = np.meshgrid(np.arange(ho), np.arange(sh.W * sh.Fh), indexing="ij")
    k, u = e // sh.Fh, e % sh.Fh
    expect = x[:, :, m * sh.s + u, k]
    assert np.array_equal(xhat, expect)
    # it is a pure copy: multiset of values is a sub-multiset of the input's
    assert np.isin(xhat, x).all()


@pytest.mark.parametrize("dims", TINY_SHAPES)
def test_im2win_row_overlap(dims):
    """Section III-A: for Hf > s the lower Hf-s rows of window row m are the upper rows of window row m+1."""
    sh = Shape(*dims)
    x = _rand((sh.N, sh.C, sh.H, sh.W), 12)
    xhat = oracle.im2win(x, sh)
    ho, _ = oracle.out_dims(sh)
    v = xhat.reshape(sh.N, sh.C, ho, sh.W, sh.Fh)
    if sh.Fh > sh.s and ho > 1:
        assert np.array_equal(v[:, :, :-1, :, sh.s:], v[:, :, 1:, :, :sh.Fh - sh.s])
    # each strip viewed as (W, Fh) is the transposed Fh x W slab of the input
    for m in range(ho):
        assert np.array_equal(v[:, :, m].transpose(0, 1, 3, 2), x[:, :, m * sh.s:m * sh.s + sh.Fh, :])


def test_im2win_identity_for_1x1():
    sh = Shape(2, 3, 6, 5, 2, 1, 1, 1)
    x = _rand((2, 3, 6, 5), 13)
    assert np.array_equal(oracle.im2win(x, sh).reshape(x.shape), x)


# ---------------------------------------------------------------- convolution routes agree
@pytest.mark.parametrize("dims", TINY_SHAPES)
def test_three_routes_agree(dims):
    sh = Shape(*dims)
    x = _rand((sh.N, sh.C, sh.H, sh.W), 21)
    f = _rand((sh.K, sh.C, sh.Fh, sh.Fw), 22)
    r1 = oracle.conv_direct(x, f, sh)
    r3 = oracle.conv_via_im2win(oracle.im2win(x, sh), f, sh)
    r4, _ = oracle.conv_via_im2col(x, f, sh)
    scale = np.abs(r1).max() + 1e-30
    assert np.abs(r1 - r3).max() / scale < 1e-12
    assert np.abs(r1 - r4).max() / scale < 1e-12


@pytest.mark.parametrize("dims", TINY_SHAPES)
def test_conv_matches_library_conv2d(dims):
    """torch's fp64 conv2d is an independent implementation of valid strided cross-correlation."""
    sh = Shape(*dims)
    x = _rand((sh.N, sh.C, sh.H, sh.W), 31)
    f = _rand((sh.K, sh.C, sh.Fh, sh.Fw), 32)
    ref = torch.nn.functional.conv2d(torch.from_numpy(x).double(), torch.from_numpy(f).double(),
                                     stride=sh.s).numpy()
    for got in (oracle.conv_direct(x, f, sh), oracle.conv_via_im2win(oracle.im2win(x, sh), f, sh)):
        assert got.shape == ref.shape
        assert np.abs(got - ref).max() / (np.abs(ref).max() + 1e-30) < 1e-12


def test_conv_matches_library_on_tiny_config():
    l = wl.CONFIGS["tiny"]
    sh = Shape(*l.dims())
    x, f = wl.make_input(l), wl.make_filter(l)
    ref = torch.nn.functional.conv2d(torch.from_numpy(x).double(), torch.from_numpy(f).double(), stride=l.s).numpy()
    got = oracle.conv_direct(x, f, sh)
    assert got.shape == (1, 16, 30, 30)
    assert np.abs(got - ref).max() < 1e-12
    # unfold is the library's im2col: same element count as the oracle's im2col count
    cols = torch.nn.functional.unfold(torch.from_numpy(x), (l.Fh, l.Fw), stride=l.s)
    assert cols.numel() == oracle.counts(sh)["im2col"] == 24300
    assert oracle.counts(sh)["im2win"] == 8640


def test_conv_bruteforce_python_loops():
    """Direct definition, pure Python, on a case small enough to loop over."""
    sh = Shape(1, 2, 5, 6, 2, 2, 3, 2)
    x = _rand((1, 2, 5, 6), 41).astype(np.float64)
    f = _rand((2, 2, 2, 3), 42).astype(np.float64)
    ho, wo = oracle.out_dims(sh)
    exp = np.zeros((1, 2, ho, wo))
    for j, m, n, r, u, v in itertools.product(range(2), range(ho), range(wo), range(2), range(2), range(3)):
        exp[0, j, m, n] += x[0, r, m * 2 + u, n * 2 + v] * f[j, r, u, v]
    for got in (oracle.conv_direct(x, f, sh), oracle.conv_via_im2win(oracle.im2win(x, sh), f, sh)):
        assert np.abs(got - exp).max() < 1e-12


# ---------------------------------------------------------------- textbook special cases
def test_special_1x1_is_per_pixel_matvec():
    sh = Shape(2, 5, 4, 3, 6, 1, 1, 1)
    x, f = _rand((2, 5, 4, 3), 51), _rand((6, 5, 1, 1), 52)
    exp = np.einsum("kc,nchw->nkhw", f[:, :, 0, 0].astype(np.float64), x.astype(np.float64))
    assert np.abs(oracle.conv_direct(x, f, sh) - exp).max() < 1e-12
    assert np.abs(oracle.conv_via_im2win(oracle.im2win(x, sh), f, sh) - exp).max() < 1e-12


def test_special_full_size_filter_is_matrix_vector_product():
    sh = Shape(3, 2, 4, 5, 3, 4, 5, 1)
    x, f = _rand((3, 2, 4, 5), 53), _rand((3, 2, 4, 5), 54)
    exp = (f.reshape(3, -1).astype(np.float64) @ x.reshape(3, -1).astype(np.float64).T).T
    for got in (oracle.conv_direct(x, f, sh), oracle.conv_via_im2win(oracle.im2win(x, sh), f, sh)):
        assert got.shape == (3, 3, 1, 1)
        assert np.abs(got[:, :, 0, 0] - exp).max() < 1e-12


@pytest.mark.parametrize("dims", [(2, 3, 9, 10, 2, 3, 2, 2), (1, 2, 8, 8, 2, 2, 3, 1), (1, 3, 12, 11, 2, 3, 3, 3)])
def test_special_one_hot_filter_is_strided_crop(dims):
    """A filter that is 1 at (r0,u0,v0) and 0 elsewhere returns I[i][r0][m*s+u0][n*s+v0]; any wrong
    sign, dropped term, swapped u/v or transposed operand moves or scales the crop."""
    sh = Shape(*dims)
    x = _rand((sh.N, sh.C, sh.H, sh.W), 55)
    ho, wo = oracle.out_dims(sh)
    for r0, u0, v0 in itertools.product(range(sh.C), range(sh.Fh), range(sh.Fw)):
        f = np.zeros((sh.K, sh.C, sh.Fh, sh.Fw), np.float32)
        f[0, r0, u0, v0] = 1.0
        f[1, r0, u0, v0] = -2.0
        crop = x[:, r0, u0:u0 + (ho - 1) * sh.s + 1:sh.s, v0:v0 + (wo - 1) * sh.s + 1:sh.s].astype(np.float64)
        for got in (oracle.conv_direct(x, f, sh), oracle.conv_via_im2win(oracle.im2win(x, sh), f, sh)):
            assert np.array_equal(got[:, 0], crop)
            assert np.array_equal(got[:, 1], -2.0 * crop)


def test_special_all_ones():
    sh = Shape(2, 3, 7, 6, 2, 3, 2, 2)
    x, f = np.ones((2, 3, 7, 6), np.float32), np.ones((2, 3, 3, 2), np.float32)
    assert np.all(oracle.conv_direct(x, f, sh) == 3 * 3 * 2)
    assert np.all(oracle.conv_via_im2win(oracle.im2win(x, sh), f, sh) == 18)


def test_linearity_and_channel_additivity():
    sh = Shape(1, 3, 8, 8, 2, 3, 3, 1)
    x, y, f = _rand((1, 3, 8, 8), 61), _rand((1, 3, 8, 8), 62), _rand((2, 3, 3, 3), 63)
    # exact in double for inputs that are sums of fp32 values held in fp32: use ints
    xi, yi, fi = np.round(x * 8), np.round(y * 8), np.round(f * 8)
    a = oracle.conv_direct((xi + yi).astype(np.float32), fi, sh)
    b = oracle.conv_direct(xi, fi, sh) + oracle.conv_direct(yi, fi, sh)
    assert np.array_equal(a, b)
    per_channel = sum(oracle.conv_direct(xi[:, c:c + 1], fi[:, c:c + 1], Shape(1, 1, 8, 8, 2, 3, 3, 1)) for c in range(3))
    assert np.array_equal(oracle.conv_direct(xi, fi, sh), per_channel)


# ---------------------------------------------------------------- sampled-point route and argument checks
def test_points_route_equals_full():
    sh = Shape(2, 3, 9, 10, 4, 3, 3, 2)
    x, f = _rand((2, 3, 9, 10), 71), _rand((4, 3, 3, 3), 72)
    full = oracle.conv_direct(x, f, sh)
    ho, wo = oracle.out_dims(sh)
    idx = np.array(list(itertools.product(range(2), range(4), range(ho), range(wo))), dtype=np.int32)
    assert np.array_equal(oracle.conv_direct_points(x, f, sh, idx), full.reshape(-1))
    with pytest.raises(ValueError):
        oracle.conv_direct_points(x, f, sh, np.array([[0, 0, ho, 0]], np.int32))


def test_rejects_bad_shapes():
    for bad in [Shape(0, 1, 4, 4, 1, 2, 2, 1), Shape(1, 1, 4, 4, 1, 5, 2, 1), Shape(1, 1, 4, 4, 1, 2, 2, 0)]:
        with pytest.raises(ValueError):
            oracle.out_dims(bad)


def test_stride_larger_than_filter_is_accepted():
    sh = Shape(1, 2, 11, 11, 2, 2, 2, 4)
    x, f = _rand((1, 2, 11, 11), 81), _rand((2, 2, 2, 2), 82)
    ref = torch.nn.functional.conv2d(torch.from_numpy(x).double(), torch.from_numpy(f).double(), stride=4).numpy()
    assert np.abs(oracle.conv_via_im2win(oracle.im2win(x, sh), f, sh) - ref).max() < 1e-12
    assert oracle.counts(sh)["im2win"] < oracle.counts(sh)["input"]
