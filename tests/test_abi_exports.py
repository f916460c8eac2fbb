"""The C-ABI library builds, loads and exports every symbol the header declares (no GPU, no compute)."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "knnssd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(knnssd_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    from paper_2505_16162_b200 import build
    lib = ctypes.CDLL(build.build())
    names = _declared()
    assert len(names) >= 14
    for n in names:
        assert hasattr(lib, n), f"{n} declared in include/knnssd.h but not exported"


def test_binding_names_match_the_header():
    from paper_2505_16162_b200 import build
    build.build()
    from paper_2505_16162_b200 import binding
    assert sorted(binding.EXPORTS) == _declared()


def test_null_arguments_are_rejected_without_a_gpu():
    from paper_2505_16162_b200 import build
    lib = ctypes.CDLL(build.build())
    lib.knnssd_init.restype = ctypes.c_int
    assert lib.knnssd_init(None, None, None, None, None, None) == 1
    lib.knnssd_get_length.restype = ctypes.c_int
    assert lib.knnssd_get_length(None) == -1
    lib.knnssd_last_error.restype = ctypes.c_char_p
    assert lib.knnssd_last_error(None) == b"NULL context"
    lib.knnssd_linear.restype = ctypes.c_int
    assert lib.knnssd_linear(None, 0, 1, 8, None, 1, None, None) == 1
