"""CPU-side checks of the boundary: the library builds, loads without a GPU and exports
every function the header declares; the binding names the same functions."""
import ctypes
import os
import re

from paper_2605_23163_b200 import build, fdd

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "fdd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(fdd_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    build.build_library()
    lib = ctypes.CDLL(fdd.LIB_PATH)
    names = _declared()
    assert len(names) >= 13
    for n in names:
        assert hasattr(lib, n), n


def test_binding_covers_header():
    assert sorted(fdd.EXPORTS) == _declared()
    for n in fdd.EXPORTS:
        assert callable(getattr(fdd, n)), n


def test_status_codes_match_header():
    text = open(os.path.join(ROOT, "include", "fdd.h")).read()
    for name, val in re.findall(r"#define\s+(FDD_[A-Z_0-9]+)\s+\(?(-?\d+)\)?", text):
        assert getattr(fdd, name) == int(val), name
