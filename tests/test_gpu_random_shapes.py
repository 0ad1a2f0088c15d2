"""Seeded random shapes through the kernel configurations, on small-integer data, bit for bit against the
oracle's Eq. (1): the fixed shape lists of the other files are hand-picked corner cases; these draws reach
combinations nobody picked (tile counts, ragged tails, channel and filter counts, strides, filter sizes)."""
import random

import numpy as np
import pytest

from paper_2306_14320_b200 import binding as b
from paper_2306_14320_b200 import workloads as wl
from gpu_helpers import apply_config, ensure_built, gpu_conv, oracle_conv, reset_config
from test_gpu_nhwc import gpu_conv_nhwc

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


def _deep_shapes(seed, count):
    """Shapes the strip-matrix and window-offset kernels take: 3x3 / 5x5, channels in multiples of 16."""
    rng = random.Random(seed)
    out = []
    while len(out) < count:
        f = rng.choice([3, 3, 3, 5])
        s = rng.choice([1, 1, 1, 2]) if f == 3 else 1
        c = rng.choice([16, 32, 64, 96, 128, 160, 256, 384])
        k = rng.choice([8, 24, 32, 64, 100, 128, 144, 192, 256, 288, 320, 384, 512])
        h, w, n = rng.randint(f, 48), rng.randint(f, 100), rng.randint(1, 6)
        if n * c * h * w * k <= 2e9:
            out.append((n, c, h, w, k, f, f, s))
    return out


def _general_shapes(seed, count):
    """Any filter size, stride and channel count (persistent specialisations, generic kernel)."""
    rng = random.Random(seed)
    out = []
    for _ in range(count):
        fh = rng.choice([1, 2, 3, 3, 5, 7, 11])
        fw = fh if rng.random() < 0.7 else rng.choice([1, 2, 3, 4, 5])
        s = rng.choice([1, 1, 2, 3, 4])
        c = rng.choice([1, 3, 4, 7, 8, 12, 16, 24, 40, 64, 100])
        k = rng.choice([1, 5, 16, 17, 64, 96, 130, 256, 300])
        out.append((rng.randint(1, 5), c, rng.randint(fh, 60), rng.randint(fw, 120), k, fh, fw, s))
    return out


DEEP = _deep_shapes(2306, 40)
GENERAL = _general_shapes(14320, 40)
DEEP_CONFIGS = ["auto", "window", "window1", "wtwo", "wstream", "wpair", "wpair2", "strip", "strip2", "pair", "pair2", "nostrip"]
GENERAL_CONFIGS = ["auto", "minws", "nostrip", "nobox", "nopim", "split3", "bslice", "generic"]


@pytest.fixture(scope="module", autouse=True)
def _built():
    ensure_built()


def _check(dims, configs, modes, seed):
    n, c, h, w, k, fh, fw, s = dims
    x = wl.small_ints(seed, n * c * h * w).reshape(n, c, h, w)
    f = wl.small_ints(seed + 1, k * c * fh * fw, -2, 2).reshape(k, c, fh, fw)
    ref = oracle_conv(x, f, dims)
    for cfg in configs:
        for mode in modes:
            for src in (b.SRC_NCHW, b.SRC_NCHW_FUSED):
                apply_config(cfg)
                try:
                    got = gpu_conv(x, f, dims, mode, src_kind=src)
                    assert np.array_equal(got.astype(np.float64), ref), (dims, cfg, mode, src)
                    if src == b.SRC_NCHW and cfg in ("auto", "window", "wpair2", "nostrip", "generic"):
                        nhwc = gpu_conv_nhwc(x, f, dims, mode, src)
                        assert np.array_equal(np.transpose(nhwc, (0, 3, 1, 2)).astype(np.float64), ref), (dims, cfg, mode, "nhwc")
                finally:
                    reset_config()


@pytest.mark.parametrize("dims", DEEP, ids=lambda d: "x".join(map(str, d)))
def test_random_deep_shapes_bit_exact(dims):
    _check(dims, DEEP_CONFIGS, (b.MODE_TF32, b.MODE_BF16), 7000 + sum(dims))


@pytest.mark.parametrize("dims", GENERAL, ids=lambda d: "x".join(map(str, d)))
def test_random_general_shapes_bit_exact(dims):
    _check(dims, GENERAL_CONFIGS, (b.MODE_TF32, b.MODE_BF16, b.MODE_FP32), 9000 + sum(dims))
