"""The C-ABI library builds, loads without a GPU and exports every function include/dat.h declares."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "dat.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dat_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    from paper_2206_06257_b200 import build
    lib = ctypes.CDLL(build.build())
    names = _declared()
    assert "dat_step" in names and "dat_quantize" in names and len(names) >= 12
    for n in names:
        assert hasattr(lib, n), n


def test_binding_lists_the_same_names():
    from paper_2206_06257_b200 import api
    assert sorted(api.EXPORTS) == _declared()
    for n in api.EXPORTS:
        assert callable(getattr(api, n))


def test_strerror_and_cpu_side_validation():
    from paper_2206_06257_b200 import api
    for code in range(-8, 1):
        assert api.dat_strerror(code) and "unknown" not in api.dat_strerror(code)
    assert "unknown" in api.dat_strerror(-99)
    # layout faults are reported before any CUDA call, so this works without a GPU
    for offs, code in (([1, 5], api.DAT_ERR_LAYOUT), ([0, 5, 5], api.DAT_ERR_LAYOUT), ([0, 4, 2], api.DAT_ERR_LAYOUT)):
        try:
            api.dat_plan_create(offs, 2, 8)
            assert False
        except api.DatError as e:
            assert e.code == code
    assert api.dat_plan_sizes.__doc__
