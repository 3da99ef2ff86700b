"""The C-ABI library builds, loads and exports every symbol that include/*.h declares.
No compute call is made here (no GPU needed)."""
import ctypes
import glob
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib_path():
    from paper_2508_13478_b200 import build
    return build.build()


def declared_symbols():
    names = []
    for path in sorted(glob.glob(os.path.join(ROOT, "include", "*.h"))):
        text = re.sub(r"/\*.*?\*/", "", open(path).read(), flags=re.S)
        names += re.findall(r"DHQ(?:_PEAKS)?_API\s+[^;{]*?\b(dhq_\w+)\s*\(", text)
    return names


def test_headers_declare_the_expected_entry_points():
    names = declared_symbols()
    for must in ("dhq_prepare", "dhq_forward", "dhq_calibrate", "dhq_forward_debug", "dhq_get_layer",
                 "dhq_last_status", "dhq_destroy", "dhq_status_string", "dhq_forward_host", "dhq_measure_pipe"):
        assert must in names
    assert len(names) == len(set(names))


def test_library_exports_every_declared_symbol(lib_path):
    lib = ctypes.CDLL(lib_path)
    for name in declared_symbols():
        assert hasattr(lib, name), f"{name} is declared in include/ but not exported"


def test_status_strings_and_binding_load(lib_path):
    import paper_2508_13478_b200 as dhq
    assert dhq.library_path() == lib_path
    assert dhq.dhq_status_string(0) == "ok"
    assert "unsupported" in dhq.dhq_status_string(2)
    assert dhq.dhq_status_string(6) != dhq.dhq_status_string(5)


def test_oracle_and_product_do_not_import_each_other():
    for path in glob.glob(os.path.join(ROOT, "oracle", "*.py")) + glob.glob(os.path.join(ROOT, "oracle", "*.c")):
        assert "paper_2508_13478_b200" not in open(path).read()
    for base, _, files in os.walk(os.path.join(ROOT, "paper_2508_13478_b200")):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(base, f)).read()
                assert "oracle" not in text.lower(), f"{f} mentions the oracle"
