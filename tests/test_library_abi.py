"""The C-ABI library loads without a GPU and exports every function include/ngalore.h declares."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "ngalore.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = set(re.findall(r"\b(ngalore_[a-z_0-9]+)\s*\(", text))
    assert len(names) >= 15
    return sorted(names)


def test_library_exports_every_declared_symbol():
    import __graft_entry__ as entry

    entry.build()
    lib = ctypes.CDLL(os.path.join(ROOT, "paper_2410_16029_b200", "libngalore.so"))
    for name in _declared_functions():
        assert hasattr(lib, name), f"{name} is declared in ngalore.h but not exported"


def test_host_side_argument_checks_need_no_device():
    import __graft_entry__ as entry

    entry.build()
    lib = ctypes.CDLL(os.path.join(ROOT, "paper_2410_16029_b200", "libngalore.so"))
    lib.ngalore_status_string.restype = ctypes.c_char_p
    assert lib.ngalore_status_string(0) == b"ok"
    assert b"Cholesky" in lib.ngalore_status_string(6)
    out = ctypes.c_void_p()
    # null shapes / non-positive counts are rejected before any CUDA call
    assert lib.ngalore_create(None, 0, 8, 4, 10, ctypes.c_double(1e-3), ctypes.c_double(1e-3), ctypes.c_double(0.9),
                              ctypes.c_double(0.999), ctypes.c_double(1e-8), ctypes.c_double(0.0), None,
                              ctypes.byref(out)) == 1
    assert lib.ngalore_step(None, None, None, None) == 1
    assert lib.ngalore_rank(None, 0) == -1
    lib.ngalore_destroy(None)
