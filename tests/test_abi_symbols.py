"""The C-ABI library loads without a GPU and exports every function include/rt3d.h declares."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "rt3d.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = re.findall(r"\b(rt3d_[a-z0-9_]+)\s*\(", text)
    return sorted(set(names))


def test_library_exports_every_declared_symbol():
    from paper_2007_09835_b200 import build
    lib = ctypes.CDLL(build.build())
    names = _declared_functions()
    assert len(names) >= 15
    for n in names:
        assert hasattr(lib, n), f"{n} declared in rt3d.h but not exported"


def test_status_strings_and_version():
    import paper_2007_09835_b200 as rt3d
    assert "sm_100a" in rt3d.rt3d_version()
    for code in range(8):
        assert rt3d.lib().rt3d_status_string(code)
    assert rt3d.rt3d_launch_count() >= 0
