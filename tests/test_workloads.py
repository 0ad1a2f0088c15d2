"""The synthetic-input module: reproducible, range-independent, distributions and zero border as stated."""
import numpy as np

from paper_2306_14320_b200 import workloads as wl


def test_streams_are_reproducible_and_counter_based():
    a, b = wl.normal01(7, 1000), wl.normal01(7, 2000)
    assert np.array_equal(a, b[:1000])
    assert not np.array_equal(wl.normal01(8, 1000), a)
    u = wl.uniform01(3, 100000)
    assert u.min() >= 0.0 and u.max() < 1.0 and abs(u.mean() - 0.5) < 0.01
    n = wl.normal01(3, 200000)
    assert abs(n.mean()) < 0.01 and abs(n.std() - 1.0) < 0.01
    i = wl.small_ints(5, 10000)
    assert set(np.unique(i)) == set(float(v) for v in range(-4, 5))


def test_sub_batch_matches_full_batch():
    l = wl.CONFIGS["resnet3x3"].with_batch(4)
    full = wl.make_input(l)
    assert np.array_equal(wl.make_input(l, slice(1, 3)), full[1:3])
    assert np.array_equal(wl.make_input(wl.CONFIGS["resnet3x3"], slice(1, 3)), full[1:3])


def test_zero_border_and_scales():
    l = wl.CONFIGS["resnet3x3"].with_batch(2)
    x, f = wl.make_input(l), wl.make_filter(l)
    assert x.shape == (2, 64, 58, 58) and f.shape == (64, 64, 3, 3)
    assert not x[:, :, 0].any() and not x[:, :, -1].any() and not x[:, :, :, 0].any() and not x[:, :, :, -1].any()
    assert abs(x[:, :, 1:-1, 1:-1].std() - 1.0) < 0.01
    assert abs(f.std() / np.sqrt(2.0 / (64 * 9)) - 1.0) < 0.02
    s = wl.CONFIGS["stem7x7"].with_batch(1)
    xs = wl.make_input(s)
    assert not xs[:, :, :3].any() and xs[:, :, 3:-3, 3:-3].min() >= 0.0 and xs.max() < 1.0
    t = wl.CONFIGS["tiny"]
    xt = wl.make_input(t)
    assert xt.shape == (1, 3, 32, 32) and xt.min() >= -1.0 and xt.max() < 1.0 and xt.min() < -0.9


def test_named_configs_cover_the_benchmark_definition():
    assert [wl.CONFIGS[k].dims() for k in ("tiny", "resnet3x3", "stem7x7", "deep3x3", "down3x3")] == [
        (1, 3, 32, 32, 16, 3, 3, 1), (128, 64, 58, 58, 64, 3, 3, 1), (128, 3, 230, 230, 64, 7, 7, 2),
        (128, 256, 16, 16, 256, 3, 3, 1), (128, 128, 58, 58, 256, 3, 3, 2)]
    assert len(wl.SWEEP) == 12 and wl.SWEEP[8].dims() == wl.CONFIGS["resnet3x3"].dims()
    assert [l.dims()[1:] for l in wl.TABLE_I_LAYERS] == [(c, h, h, k, f, f, s) for c, h, k, f, s in wl.TABLE_I]
