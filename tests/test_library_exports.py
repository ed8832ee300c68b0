"""The built C-ABI library loads and exports every symbol the public header declares (no GPU needed)."""
import ctypes
import os
import re

from paper_2602_16052_b200 import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "moespec.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(moespec_[a-z_]+)\s*\(", text)))


def test_library_builds_and_exports_header_symbols():
    path = build.build()
    lib = ctypes.CDLL(path)
    names = declared_symbols()
    assert "moespec_layer_create" in names and "moespec_verify_layer" in names and "moespec_destroy" in names
    for n in names:
        assert hasattr(lib, n), n
    lib.moespec_strerror.restype = ctypes.c_char_p
    assert lib.moespec_strerror(0) == b"ok"
    assert lib.moespec_version() >= 100
    assert lib.moespec_destroy(None) == 0            # NULL is accepted
    assert lib.moespec_layer_create(None, None) == -2


def test_binding_lists_every_export():
    from paper_2602_16052_b200 import moespec
    assert sorted(moespec.EXPORTS) == declared_symbols()
