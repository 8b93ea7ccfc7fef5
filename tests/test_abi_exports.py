"""CPU-only: the C-ABI library builds, loads, and exports every symbol include/snlp.h declares."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "snlp.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(snlp_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    from paper_2605_17842_b200 import build
    path = build.build()
    lib = ctypes.CDLL(path)
    names = declared_functions()
    assert len(names) >= 15
    for n in names:
        assert hasattr(lib, n), n


def test_binding_lists_the_same_entry_points():
    from paper_2605_17842_b200 import build
    build.build()
    from paper_2605_17842_b200 import snlp
    assert sorted(snlp.EXPORTS) == declared_functions()


def test_header_has_no_torch_or_cxx_types():
    text = open(os.path.join(ROOT, "include", "snlp.h")).read()
    assert "torch" not in text and "std::" not in text and "at::" not in text
