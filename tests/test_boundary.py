"""Host-side checks of the C-ABI boundary that need no GPU: the library loads, exports every symbol the
header declares, answers the size queries like the oracle's closed forms, and rejects bad arguments
before anything is launched."""
import ctypes
import os
import re

import pytest

import oracle
from paper_2306_14320_b200 import binding as b
from paper_2306_14320_b200 import build, workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build_library()


def _declared():
    names = []
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names += re.findall(r"\b(im2win_[a-z0-9_]+)\s*\(", text)
    return sorted(set(names))


def test_library_exports_every_declared_symbol():
    declared = _declared()
    assert set(declared) == set(b.EXPORTS)
    L = ctypes.CDLL(b.LIB_PATH)
    for name in declared:
        assert getattr(L, name) is not None


def test_size_queries_match_closed_forms():
    layers = [l.dims() for l in wl.CONFIGS.values()] + [(128, c, h, h, k, f, f, s) for c, h, k, f, s in wl.TABLE_I]
    layers += [(1, 1, 4, 4, 1, 2, 2, 1), (2, 3, 9, 11, 2, 2, 3, 4), (1, 2, 8, 8, 2, 2, 2, 2)]
    for d in layers:
        c = oracle.counts(oracle.Shape(*d))
        assert b.out_dims(d) == oracle.out_dims(oracle.Shape(*d))
        assert b.workspace_bytes(d) == 4 * c["im2win"]
        assert b.im2col_bytes(d) == 4 * c["im2col"]
    # the paper's illustration: 24 vs 36 elements
    assert (b.workspace_bytes((1, 1, 4, 4, 1, 2, 2, 1)), b.im2col_bytes((1, 1, 4, 4, 1, 2, 2, 1))) == (96, 144)
    # Table I Conv4 is large: sizes are 64-bit
    assert b.workspace_bytes((128, 64, 224, 224, 64, 7, 7, 2)) == 4 * 128 * 64 * 109 * 7 * 224


@pytest.mark.parametrize("dims", [(0, 1, 4, 4, 1, 2, 2, 1), (1, 1, 4, 4, 1, 5, 2, 1), (1, 1, 4, 4, 1, 2, 5, 1),
                                  (1, 1, 4, 4, 1, 2, 2, 0), (1, 1, 4, 4, 0, 2, 2, 1), (1, -3, 4, 4, 1, 2, 2, 1),
                                  (2 ** 31 - 1, 2 ** 31 - 1, 2 ** 31 - 1, 2 ** 31 - 1, 1, 1, 1, 1)])
def test_bad_shapes_are_einval(dims):
    for fn in (b.out_dims, b.workspace_bytes, b.im2col_bytes):
        with pytest.raises(b.Im2winError) as e:
            fn(dims)
        assert e.value.code == b.EINVAL


def test_argument_checks_happen_before_any_launch():
    d = (1, 3, 32, 32, 16, 3, 3, 1)
    A, B_, C_, D = 0x10000000, 0x20000000, 0x30000000, 0x40000000  # never dereferenced: the checks fail first
    cases = [
        (lambda: b.transform(0, d, B_, stream=0), b.EINVAL),
        (lambda: b.transform(A, d, 0, stream=0), b.EINVAL),
        (lambda: b.transform(A + 4, d, B_, stream=0), b.EALIGN),
        (lambda: b.transform(A, d, B_ + 8, stream=0), b.EALIGN),
        (lambda: b.transform(A, d, A + 1024, stream=0), b.EOVERLAP),
        (lambda: b.conv(A, b.SRC_NCHW, B_, d, b.MODE_TF32, C_, None, 0, stream=0), b.EWORKSPACE),
        (lambda: b.conv(A, b.SRC_NCHW, B_, d, b.MODE_TF32, C_, D, b.workspace_bytes(d) - 4, stream=0), b.EWORKSPACE),
        (lambda: b.conv(A, 7, B_, d, b.MODE_TF32, C_, D, 1 << 20, stream=0), b.EINVAL),
        (lambda: b.conv(A, b.SRC_IM2WIN, B_, d, 9, C_, None, 0, stream=0), b.EINVAL),
        (lambda: b.conv(A, b.SRC_IM2WIN, B_ + 2, d, b.MODE_BF16, C_, None, 0, stream=0), b.EALIGN),
        (lambda: b.conv(A, b.SRC_IM2WIN, B_, d, b.MODE_BF16, A + 64, None, 0, stream=0), b.EOVERLAP),
        (lambda: b.conv(A, b.SRC_NCHW, B_, d, b.MODE_BF16, C_, C_ + 16, 1 << 20, stream=0), b.EOVERLAP),
        (lambda: b.conv(0, b.SRC_IM2WIN, B_, d, b.MODE_BF16, C_, None, 0, stream=0), b.EINVAL),
    ]
    for call, code in cases:
        with pytest.raises(b.Im2winError) as e:
            call()
        assert e.value.code == code, (code, e.value)


def test_static_scratch_constant_matches_header():
    text = open(os.path.join(ROOT, "include", "im2win.h")).read()
    m = re.search(r"#define\s+IM2WIN_STATIC_SCRATCH_BYTES\s+\((\d+)u \* (\d+)u \* (\d+)u\)", text)
    assert m and int(m.group(1)) * int(m.group(2)) * int(m.group(3)) == b.STATIC_SCRATCH_BYTES


def test_strerror_covers_every_code():
    texts = {b.strerror(c) for c in range(0, -10, -1)}
    assert len(texts) == 10 and all(texts)


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(b, "_lib", None)
    monkeypatch.setattr(b, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(ImportError):
        b.out_dims((1, 1, 4, 4, 1, 2, 2, 1))
    monkeypatch.setattr(b, "_lib", None)
