"""The C-ABI library loads without a GPU and exports every symbol include/bigbird.h declares."""
import ctypes
import os
import re

import paper_2007_14062_b200 as bb

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    names = []
    for fn in sorted(os.listdir(os.path.join(ROOT, "include"))):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            names += re.findall(r"BIGBIRD_API\s+[\w\s\*]+?\b(bigbird_\w+)\s*\(", text)
    return names


def test_library_exports_every_declared_symbol():
    names = _declared()
    assert len(names) >= 11 and "bigbird_attn_fwd" in names and "bigbird_build_layout" in names
    lib = ctypes.CDLL(bb.library_path())
    for n in names:
        assert hasattr(lib, n), n


def test_binding_has_the_same_names():
    for n in ("bigbird_build_layout", "bigbird_attn_fwd", "bigbird_attn_fwd_simt", "bigbird_last_status", "bigbird_strerror"):
        assert callable(getattr(bb, n))


def test_no_oracle_import_in_the_package():
    pkg = os.path.join(ROOT, "paper_2007_14062_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cpp", ".h", ".cuh")):
                text = open(os.path.join(dirpath, f)).read()
                assert not re.search(r"^\s*(from|import)\s+oracle\b|oracle[/.]bigbird_oracle|#include.*oracle", text,
                                     flags=re.M), os.path.join(dirpath, f)
