"""The C-ABI library: it loads without a GPU, exports every function include/dart.h declares, and the
binding refuses to work without it.  No compute calls.  CPU only."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def built():
    from paper_2502_11494_b200 import build

    return build.build_library()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "dart.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dart_[a-z_0-9]+)\s*\(", text)))


def test_header_functions_are_exported(built):
    names = declared_functions()
    assert "dart_reduce" in names and "dart_create" in names and len(names) >= 12
    L = ctypes.CDLL(built)
    for n in names:
        assert hasattr(L, n), "libdart.so does not export %s" % n


def test_binding_lists_the_same_entry_points(built):
    from paper_2502_11494_b200 import dart

    assert sorted(dart.EXPORTS) == declared_functions()
    for n in dart.EXPORTS:
        assert callable(getattr(dart, n))
    assert dart.dart_version() == 100
    assert "NULL" in dart.dart_strerror(dart.DART_ERR_NULL)


def test_struct_layouts_match_the_header():
    from paper_2502_11494_b200 import dart

    assert ctypes.sizeof(dart.dart_desc) == 28
    assert ctypes.sizeof(dart.dart_opts) == 88 and dart.dart_opts.pivots_in.offset == 40 and dart.dart_opts.cu_seqlens.offset == 48
    assert dart.dart_opts.resident_split.offset == 56 and dart.dart_opts.seed.offset == 72 and dart.dart_opts.tune.offset == 84
    assert ctypes.sizeof(dart.dart_debug) == 7 * ctypes.sizeof(ctypes.c_void_p)


def test_binding_constants_equal_the_header_defines():
    """Every numeric DART_* #define of the header that the binding names has the same value there."""
    from paper_2502_11494_b200 import dart

    text = open(os.path.join(ROOT, "include", "dart.h")).read()
    defines = {m.group(1): int(m.group(2), 0) for m in re.finditer(r"^#define\s+(DART_[A-Z_0-9]+)\s+\(?(-?(?:0x[0-9a-fA-F]+|\d+))\)?", text, flags=re.M)}
    assert len(defines) >= 20
    checked = 0
    for name, value in defines.items():
        if hasattr(dart, name):
            assert getattr(dart, name) == value, name
            checked += 1
    for name in ("DART_RETAIN_BANDS", "DART_RETAIN_FUSED", "DART_PATH_PAIRED", "DART_PATH_SPLIT", "DART_PIVOTS_RANDOM", "DART_RULE_UNION"):
        assert name in defines and hasattr(dart, name), name
    assert checked >= 18


def test_null_arguments_are_rejected_without_a_device(built):
    from paper_2502_11494_b200 import dart

    L = dart.lib()
    assert L.dart_create(None, None) == dart.DART_ERR_NULL
    assert dart.dart_set_shape(None, 1, 1) == dart.DART_ERR_NULL
    assert dart.dart_reduce(None, None, None, 0, 1, 1, 1, None, None, None, None) == dart.DART_ERR_NULL
    assert dart.dart_status(None) == dart.DART_ERR_NULL
    assert dart.dart_destroy(None) == dart.DART_OK
    rc, h = dart.dart_create(1, 16, 12, 1, 4)            # d not a multiple of 8
    assert rc == dart.DART_ERR_BAD_SHAPE and not h
    rc, h = dart.dart_create(1, 16, 16, 5, 4)            # more pivots than kept tokens
    assert rc == dart.DART_ERR_BAD_SHAPE


def test_no_fallback_when_library_is_missing(monkeypatch):
    from paper_2502_11494_b200 import dart

    monkeypatch.setattr(dart, "_lib", None)
    monkeypatch.setattr(dart, "LIB_PATH", os.path.join(ROOT, "does_not_exist.so"))
    with pytest.raises(RuntimeError, match="no fallback"):
        dart.dart_version()


def test_product_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2502_11494_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in src.lower() or f == "workloads.py", "%s mentions the oracle" % f
    src = open(os.path.join(pkg, "workloads.py")).read()
    assert "import oracle" not in src and "from oracle" not in src
