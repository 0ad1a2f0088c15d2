"""Seeded synthetic inputs and the named layer configurations.

This module holds no part of the im2win method: it only names problem sizes and
fills arrays with reproducible pseudo-random numbers.  Both the CPU oracle's
tests and the CUDA path's tests / benchmark draw their inputs from here, so the
two sides see identical bits without sharing any arithmetic of the method.

Generator: counter-based.  Element ``idx`` of stream ``seed`` is
``splitmix64(seed * 2**32 + idx)``; uniforms take the top 24 bits (exactly
representable in fp32), normals are Box-Muller in fp64 on two such 53-bit
uniforms and are rounded to fp32 once.  numpy only.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import numpy as np

_U64 = np.uint64


def _splitmix64(x: np.ndarray) -> np.ndarray:
    x = x.astype(np.uint64, copy=True)
    with np.errstate(over="ignore"):
        x += _U64(0x9E3779B97F4A7C15)
        z = x
        z = (z ^ (z >> _U64(30))) * _U64(0xBF58476D1CE4E5B9)
        z = (z ^ (z >> _U64(27))) * _U64(0x94D049BB133111EB)
        z = z ^ (z >> _U64(31))
    return z


def _bits(seed: int, start: int, count: int) -> np.ndarray:
    base = (int(seed) & 0xFFFFFFFF) << 32
    with np.errstate(over="ignore"):
        ctr = np.arange(start, start + count, dtype=np.uint64) + _U64(base)
    return _splitmix64(ctr)


def uniform01(seed: int, count: int) -> np.ndarray:
    """fp32 uniforms in [0, 1) with 24 random bits each."""
    return ((_bits(seed, 0, count) >> _U64(40)).astype(np.float32)) * np.float32(2.0 ** -24)


def normal01(seed: int, count: int) -> np.ndarray:
    """fp32 standard normals (Box-Muller in fp64, one rounding to fp32)."""
    out = np.empty(count, dtype=np.float32)
    chunk = 1 << 22
    for s0 in range(0, count, chunk):
        n = min(chunk, count - s0)
        b1 = _bits(seed, 2 * s0, 2 * n)
        u1 = ((b1[0::2] >> _U64(11)).astype(np.float64) + 1.0) * 2.0 ** -53  # (0, 1]
        u2 = (b1[1::2] >> _U64(11)).astype(np.float64) * 2.0 ** -53          # [0, 1)
        out[s0:s0 + n] = (np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)).astype(np.float32)
    return out


def small_ints(seed: int, count: int, lo: int = -4, hi: int = 4) -> np.ndarray:
    """fp32 integers in [lo, hi]: exactly representable in bf16, so products and short sums are exact."""
    span = hi - lo + 1
    return ((_bits(seed, 0, count) >> _U64(33)) % _U64(span)).astype(np.float32) + np.float32(lo)


@dataclass(frozen=True)
class Layer:
    """One convolution layer (valid, single stride, no bias) and the recipe for its synthetic data.

    ``H``/``W`` are the sizes actually handed to the library; ``pad`` says how many of their border
    rows/columns are an explicit ring of zeros (the caller-side padding of the named network layer).
    """
    name: str
    N: int
    C: int
    H: int
    W: int
    K: int
    Fh: int
    Fw: int
    s: int
    pad: int = 0
    input_dist: str = "normal"     # "normal" N(0,1) | "uniform01" U[0,1) | "uniform11" U[-1,1)
    filter_dist: str = "kaiming"   # "kaiming" N(0, 2/(C*Fh*Fw)) | "uniform11"
    seed: int = 0

    def dims(self) -> tuple:
        return (self.N, self.C, self.H, self.W, self.K, self.Fh, self.Fw, self.s)

    def with_batch(self, n: int) -> "Layer":
        return replace(self, N=n)


def _draw(dist: str, seed: int, count: int, fan_in: int) -> np.ndarray:
    if dist == "normal":
        return normal01(seed, count)
    if dist == "uniform01":
        return uniform01(seed, count)
    if dist == "uniform11":
        return uniform01(seed, count) * np.float32(2.0) - np.float32(1.0)
    if dist == "kaiming":
        return normal01(seed, count) * np.float32(np.sqrt(2.0 / fan_in))
    if dist == "ints":
        return small_ints(seed, count)
    raise ValueError(dist)


def make_input(layer: Layer, images: slice | None = None) -> np.ndarray:
    """Input tensor N x C x H x W (fp32).  The interior is drawn from ``layer.input_dist``; the outer
    ``pad`` rows/columns are exactly 0.  ``images`` selects a sub-range of the batch without
    generating the rest (values do not depend on the range chosen)."""
    lo, hi, _ = (images or slice(None)).indices(layer.N)
    n = max(hi - lo, 0)
    p = layer.pad
    hi_, wi_ = layer.H - 2 * p, layer.W - 2 * p
    per_img = layer.C * hi_ * wi_
    out = np.zeros((n, layer.C, layer.H, layer.W), dtype=np.float32)
    for b in range(n):
        # one stream per image keeps sub-ranges consistent with the full batch
        vals = _draw(layer.input_dist, 1000 * layer.seed + 17 + 7919 * (lo + b), per_img, 1)
        out[b, :, p:p + hi_, p:p + wi_] = vals.reshape(layer.C, hi_, wi_)
    return out


def make_filter(layer: Layer) -> np.ndarray:
    """Filter tensor K x C x Fh x Fw (fp32)."""
    fan_in = layer.C * layer.Fh * layer.Fw
    vals = _draw(layer.filter_dist, 1000 * layer.seed + 3, layer.K * fan_in, fan_in)
    return vals.reshape(layer.K, layer.C, layer.Fh, layer.Fw)


def _sweep() -> list[Layer]:
    rows = [(3, 227, 96, 11, 4), (96, 31, 256, 5, 1), (256, 15, 384, 3, 1), (384, 15, 384, 3, 1),
            (384, 15, 256, 3, 1), (3, 231, 96, 11, 4), (256, 16, 512, 3, 1), (3, 227, 64, 7, 2),
            (64, 58, 64, 3, 1), (128, 30, 128, 3, 1), (256, 16, 256, 3, 1), (512, 9, 512, 3, 1)]
    out = []
    for i, (c, h, k, f, s) in enumerate(rows, start=1):
        pad = (f - 1) // 2 if s == 1 else 0
        out.append(Layer(f"sweep_L{i}", 128, c, h, h, k, f, f, s, pad=pad, seed=50 + i))
    return out


# The named configurations of the benchmark definition.  "tiny" is the case the oracle finishes in
# well under a second; "resnet3x3" is the headline layer.
CONFIGS: dict[str, Layer] = {
    "tiny": Layer("tiny", 1, 3, 32, 32, 16, 3, 3, 1, pad=0, input_dist="uniform11",
                  filter_dist="uniform11", seed=0),
    "resnet3x3": Layer("resnet3x3", 128, 64, 58, 58, 64, 3, 3, 1, pad=1, seed=2),
    "stem7x7": Layer("stem7x7", 128, 3, 230, 230, 64, 7, 7, 2, pad=3, input_dist="uniform01", seed=3),
    "deep3x3": Layer("deep3x3", 128, 256, 16, 16, 256, 3, 3, 1, pad=1, seed=4),
    "down3x3": Layer("down3x3", 128, 128, 58, 58, 256, 3, 3, 2, pad=1, seed=5),
}
SWEEP: list[Layer] = _sweep()
for _l in SWEEP:
    CONFIGS[_l.name] = _l

def _table1() -> list[Layer]:
    return [Layer(f"table1_Conv{i}", 128, c, h, h, k, f, f, s, pad=0, seed=80 + i)
            for i, (c, h, k, f, s) in enumerate(TABLE_I, start=1)]


# The twelve layer shapes of the paper's Table I (unpadded; batch 128 in its experiments) as
# (C, H=W, K, Fh=Fw, s).  The output sizes the table prints live in tests/golden/.
TABLE_I = [(3, 227, 96, 11, 4), (3, 231, 96, 11, 4), (3, 227, 64, 7, 2), (64, 224, 64, 7, 2),
           (96, 24, 256, 5, 1), (256, 12, 512, 3, 1), (3, 224, 64, 3, 1), (64, 112, 128, 3, 1),
           (64, 56, 64, 3, 1), (128, 28, 128, 3, 1), (256, 14, 256, 3, 1), (512, 7, 512, 3, 1)]

# The same twelve as unpadded benchmark layers (batch 128, N(0,1) inputs, Kaiming-normal filters).
TABLE_I_LAYERS: list[Layer] = _table1()
for _l in TABLE_I_LAYERS:
    CONFIGS[_l.name] = _l
