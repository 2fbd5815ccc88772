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


def test_binding_constants_match_the_header():
    from paper_2510_09608_b200 import binding
    header = open(os.path.join(ROOT, "include", "svlm.h")).read()
    m = re.search(r"#define\s+SVLM_NOALLOC_SCRATCH_BYTES\s+\((\d+)u\s*<<\s*(\d+)\)", header)
    assert m and binding.NOALLOC_SCRATCH_BYTES == int(m.group(1)) << int(m.group(2))
    for name, value in re.findall(r"SVLM_(ERR_[A-Z_]+|OK)\s*=\s*(-?\d+)", header):
        assert getattr(binding, name) == int(value), name
