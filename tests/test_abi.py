"""The C-ABI library builds, loads without a GPU and exports what include/maaso.h declares."""
import ctypes
import os
import re

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "maaso.h")).read()
    return sorted(set(re.findall(r"MAASO_API[^;(]*?\b(maaso_\w+)\s*\(", text)))


def test_header_declares_the_named_entry_points():
    names = declared_functions()
    for must in ("maaso_load_profile", "maaso_load_trace", "maaso_eval_placements", "maaso_topk"):
        assert must in names


def test_library_exports_every_declared_symbol():
    import paper_2509_06362_b200 as m
    lib = ctypes.CDLL(m.lib_path())
    for name in declared_functions():
        assert hasattr(lib, name), name
        assert hasattr(m, name), f"python binding lacks {name}"


def test_layout_sizes_match_between_generators_and_binding():
    import gen
    import paper_2509_06362_b200 as m
    assert gen.REQUEST_DTYPE == m.REQUEST_DTYPE
    assert gen.SLO_DTYPE == m.SLO_DTYPE
    assert gen.RESULT_DTYPE == m.RESULT_DTYPE


def test_strerror_and_argument_checks_without_gpu():
    import paper_2509_06362_b200 as m
    assert m.maaso_strerror(0) == "ok"
    assert "invalid" in m.maaso_strerror(-1)
    lib = ctypes.CDLL(m.lib_path())
    lib.maaso_create.restype = ctypes.c_int
    assert lib.maaso_create(None, 0) == -1          # null out pointer
    assert lib.maaso_launch_count(None) == 0
    lib.maaso_destroy(None)                         # no-op


def test_product_never_imports_the_oracle():
    pkg = os.path.join(ROOT, "paper_2509_06362_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.lower(), os.path.join(dirpath, f)
