"""The shared library builds, loads without a GPU, and exports every entry point the header declares."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "vlac.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(vlac_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    from paper_2502_02175_b200 import build
    lib = ctypes.CDLL(build.build())
    names = _declared()
    assert "vlac_step" in names and "vlac_select" in names and "vlac_layer_forward" in names
    for n in names:
        assert hasattr(lib, n), n


def test_binding_lists_the_same_entry_points():
    from paper_2502_02175_b200 import build
    build.build()
    from paper_2502_02175_b200 import binding
    assert sorted(binding.EXPORTS) == _declared()
    for n in binding.EXPORTS:
        assert callable(getattr(binding, n, None)) or n == "vlac_status_string", n


def test_status_strings_need_no_device():
    from paper_2502_02175_b200 import build
    lib = ctypes.CDLL(build.build())
    lib.vlac_status_string.restype = ctypes.c_char_p
    assert lib.vlac_status_string(0) == b"ok"
    assert lib.vlac_status_string(-1) == b"invalid argument"
    assert lib.vlac_create(None, None, None) == -1
