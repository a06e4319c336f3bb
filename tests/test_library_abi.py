"""The C-ABI shared library builds, loads and exports every symbol include/dsvt.h declares. CPU only
(no compute calls)."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "dsvt.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dsvt_[a-z0-9_]+)\s*\(", text)))


def test_library_builds_loads_and_exports_declared_symbols():
    from paper_2301_06051_b200 import api, build

    path = build.build()
    assert os.path.exists(path)
    lib = ctypes.CDLL(path)
    names = _declared()
    assert len(names) >= 11
    for name in names:
        assert hasattr(lib, name), name
    assert sorted(api.EXPORTS) == names
    api.load()
    assert api.load().dsvt_error_string(0) == b"ok"
    assert api.load().dsvt_error_string(-3).startswith(b"shape")


def test_host_side_argument_errors_without_a_gpu():
    """dsvt_create refuses bad arguments before touching CUDA; a NULL context is an error everywhere."""
    from paper_2301_06051_b200 import api

    lib = api.load()
    h = ctypes.c_void_p()
    assert lib.dsvt_create(ctypes.byref(h), 0, None, 0, 1, 1) == -1
    assert lib.dsvt_create(None, 0, None, 1, 1, 1) == -1
    assert lib.dsvt_status_sync(None, None) == -1
    assert lib.dsvt_destroy(None) == 0
    g = (ctypes.c_int32 * 3)(8, 8, 1)
    assert lib.dsvt_partition(None, None, 0, 1, g, g, 3, 0, None, 0, None, None, None, None, None, None) == -1


def test_product_does_not_import_the_oracle():
    """The oracle is test infrastructure: nothing under the package may import or mention it."""
    pkg = os.path.join(ROOT, "paper_2301_06051_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text and "dsvt_ref" not in text, os.path.join(dirpath, f)
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith((".py", ".c")):
            text = open(os.path.join(ROOT, "oracle", f)).read()
            assert "paper_2301_06051_b200" not in text and "libdsvt_b200" not in text
