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


def test_contexts_share_no_mutable_state(lib):
    """Two contexts on two host threads (or two devices) must not race: the library keeps no writable
    global besides what is listed here, checked on the built image's symbol table.  The launch-attribute
    caches that used to be function-local statics are gone (the attribute is set on every launch)."""
    import subprocess
    from paper_2412_04180_b200 import skim
    out = subprocess.run(["nm", "-C", skim.LIB_PATH], capture_output=True, text=True, check=True).stdout
    allowed = (
        "skim_static_scratch",           # host-side handle of the device array of skim_quantize_static
        "g_static_ptr", "g_static_mutex",   # its per-device address cache, guarded by the mutex beside it
        "__cudaFatCubinHandle", "__fatDeviceText", "__nv_", "__cuda", "libcudart_static", "cudart",
        "completed.", "__dso_handle", "_DYNAMIC", "_GLOBAL_OFFSET_TABLE_", "__TMC_END__", "DW.ref.", "__frame_dummy",
        "__do_global_dtors", "kVariants",   # constant tables of kernel variants (relocated, hence in .data.rel.ro)
    )
    ours = []
    for line in out.splitlines():
        parts = line.split(None, 2)
        if len(parts) == 3 and parts[1] in "bBdD":
            name = parts[2]
            if any(a in name for a in allowed):
                continue
            # symbols of the statically linked CUDA runtime have hashed or internal names
            if re.fullmatch(r"[A-Za-z_][\w.]*", name) and not name.startswith("skim") and "::" not in name:
                continue
            ours.append(name)
    assert ours == [], ours


def test_two_contexts_on_two_threads_keep_their_own_settings(lib):
    """Host-side state (options, counters) lives in the context, not in the library."""
    import threading
    made = {}

    def worker(tag):
        h = C.c_void_p()
        # no device here: creation fails cleanly and leaves nothing behind, on every thread
        made[tag] = lib.skim_create(C.byref(h), C.c_int(0), C.c_void_p(0))

    ts = [threading.Thread(target=worker, args=(i,)) for i in range(2)]
    [t.start() for t in ts]
    [t.join() for t in ts]
    assert made[0] == made[1]
