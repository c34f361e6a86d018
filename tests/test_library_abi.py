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


def test_more_argument_checks_and_no_silent_success_without_a_device():
    import torch

    import __graft_entry__ as entry

    entry.build()
    lib = ctypes.CDLL(os.path.join(ROOT, "paper_2410_16029_b200", "libngalore.so"))
    d = ctypes.c_double

    class Shape(ctypes.Structure):
        _fields_ = [("rows", ctypes.c_int64), ("cols", ctypes.c_int64)]

    def create(shapes, r=8, s=4, T=10, lam=1e-3, beta1=0.9):
        arr = (Shape * max(len(shapes), 1))(*[Shape(m, n) for m, n in shapes])
        out = ctypes.c_void_p(123)
        rc = lib.ngalore_create(arr, len(shapes), r, s, T, d(lam), d(1e-3), d(beta1), d(0.999), d(1e-8), d(0.0), None,
                                ctypes.byref(out))
        return rc, out

    for bad in (dict(shapes=[]), dict(shapes=[(0, 64)]), dict(shapes=[(64, 36)]), dict(shapes=[(64, 64)], r=0),
                dict(shapes=[(64, 64)], s=33), dict(shapes=[(64, 64)], T=-1), dict(shapes=[(64, 64)], lam=0.0),
                dict(shapes=[(64, 64)], beta1=1.0), dict(shapes=[(1 << 25, 64)])):
        rc, out = create(**bad)
        assert rc == 1 and out.value is None, bad       # INVALID_ARG, and no handle is handed out
    if not torch.cuda.is_available():
        # a well-formed request without a B200 is an error too: nothing steps on the CPU instead
        rc, out = create([(64, 64)])
        assert rc != 0 and out.value is None
    # the allocation-free entry point checks its sizes on the host before it touches the device
    lib.ngalore_natural_gradient_static.argtypes = [ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_int,
                                                    ctypes.c_int, d, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                                    ctypes.c_void_p]
    fake = ctypes.c_void_p(4096)                         # never dereferenced: every call below is rejected first
    for n, s, count, cur, lam in ((8388608 + 8192, 4, 1, 0, 1e-3), (10, 4, 1, 0, 1e-3), (4096, 33, 1, 0, 1e-3),
                                  (4096, 4, 5, 0, 1e-3), (4096, 4, 2, 2, 1e-3), (4096, 4, 1, 0, 0.0)):
        assert lib.ngalore_natural_gradient_static(fake, n, s, count, cur, d(lam), fake, fake, None, None) == 1
