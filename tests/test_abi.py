"""The C-ABI library loads and exports every symbol the public header declares."""

import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    names = []
    for fn in sorted(os.listdir(os.path.join(ROOT, "include"))):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names += re.findall(r"\b(locret_[a-z0-9_]+)\s*\(", text)
    return sorted(set(names))


def test_library_exports_every_declared_symbol():
    import __graft_entry__ as G
    G.build()
    from paper_2410_01805_b200 import lib_path
    lib = ctypes.CDLL(lib_path)
    names = declared_functions()
    assert {"locret_create", "locret_prefill_chunk", "locret_decode_step", "locret_destroy"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n


def test_error_strings_and_null_handles_need_no_gpu():
    from paper_2410_01805_b200 import lib
    assert lib.locret_strerror(0) == b"ok"
    assert b"capacity" in lib.locret_strerror(-3)
    assert lib.locret_prefill_chunk(None, None, 1, 0, None) == -1
    assert lib.locret_cache_len(None, None) == -1
    lib.locret_destroy(None)


def test_product_package_does_not_touch_the_oracle():
    pkg = os.path.join(ROOT, "paper_2410_01805_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                assert "oracle" not in open(os.path.join(dirpath, f)).read(), f
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith(".py"):
            assert "paper_2410_01805_b200" not in open(os.path.join(ROOT, "oracle", f)).read()
