"""The C-ABI library loads and exports every symbol the public header declares (no GPU needed)."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    from paper_2510_09608_b200 import build
    lib = ctypes.CDLL(build.build())
    header = open(os.path.join(ROOT, "include", "svlm.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    names = set(re.findall(r"\b(svlm_[a-z_0-9]+)\s*\(", header))
    assert {"svlm_cache_create", "svlm_cache_append", "svlm_cache_evict", "svlm_attend"} <= names
    for name in sorted(names):
        assert hasattr(lib, name), name


def test_status_strings():
    from paper_2510_09608_b200 import binding
    assert binding.strerror(0) == "ok"
    for code in range(-6, 0):
        assert binding.strerror(code) != "unknown status"
