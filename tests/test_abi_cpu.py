"""CPU-only checks of the C-ABI library: it loads, exports every symbol the header declares,
and its host-only helpers (layout, sizes, messages) answer without a GPU."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2412_04180_b200 import build, skim
    build.build()
    return skim.lib()


def _declared():
    text = open(os.path.join(ROOT, "include", "skim.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(skim_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    from paper_2412_04180_b200 import skim
    names = _declared()
    assert len(names) >= 15
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(skim.EXPORTS) == names


def test_packed_layout(lib, oracle):
    from paper_2412_04180_b200.skim import Skim
    for cols in (1, 31, 32, 33, 512, 4096, 11008, 22016):
        strides, mx = Skim.packed_layout(100, cols, [1, 2, 3, 4])
        assert strides == [oracle.row_stride_words(cols, b) for b in (1, 2, 3, 4)]
        assert mx == 100 * strides[-1] * 4
    strides, _ = Skim.packed_layout(5, 100, [2, 3])
    assert strides == [oracle.row_stride_words(100, 2), oracle.row_stride_words(100, 3)]


def test_argument_errors_without_a_device(lib):
    from paper_2412_04180_b200.skim import Skim, SkimError
    with pytest.raises(SkimError) as e:
        Skim.packed_layout(10, 10, [1, 3])
    assert e.value.code == -3
    with pytest.raises(SkimError) as e:
        Skim.packed_layout(10, 10, [3, 4, 5])
    assert e.value.code == -3
    with pytest.raises(SkimError) as e:
        Skim.packed_layout(10, 0, [1, 2])
    assert e.value.code == -2
    assert Skim.workspace_bytes(4096, 11008) % 256 == 0
    assert Skim.workspace_bytes(4096, 11008) >= 296 * 11008 * 8
    assert Skim.host_staging_bytes(256, 512, [1, 2, 3, 4]) >= 256 * 512 * 6
    for code in range(-9, 1):
        assert len(lib.skim_strerror(code)) > 1
    assert lib.skim_strerror(-100) == b"unknown error"


def test_missing_library_is_a_loud_error(monkeypatch, tmp_path):
    from paper_2412_04180_b200 import skim
    monkeypatch.setattr(skim, "_lib", None)
    monkeypatch.setattr(skim, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="no fallback"):
        skim.lib()
