"""Thin ctypes binding over the C-ABI library ``libngalore.so`` (see include/ngalore.h).

Argument marshalling only: every step of the optimizer runs in the library's
CUDA kernels.  torch is used for device memory and streams.  Importing this
module fails loudly when the library has not been built; there is no fallback.
"""
from __future__ import annotations

import ctypes
import os
from typing import List, Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libngalore.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it first (python -c 'import __graft_entry__ as g; g.build()' "
        "or python -m paper_2410_16029_b200.build). There is no CPU fallback.")

_lib = ctypes.CDLL(LIB_PATH)

OK = 0
STATUS_NAMES = {0: "OK", 1: "INVALID_ARG", 2: "ALLOC", 3: "CUDA", 4: "UNSUPPORTED_DEVICE", 5: "NO_SUBSPACE",
                6: "NOT_SPD", 7: "NONFINITE", 8: "TIMEOUT"}


class Shape(ctypes.Structure):
    _fields_ = [("rows", ctypes.c_int64), ("cols", ctypes.c_int64)]


class Options(ctypes.Structure):
    _fields_ = [("struct_size", ctypes.c_int32), ("gemm_impl", ctypes.c_int32),
                ("power_iterations", ctypes.c_int32), ("reset_history_on_refresh", ctypes.c_int32),
                ("seed", ctypes.c_uint64), ("stream_impl", ctypes.c_int32), ("projection_rule", ctypes.c_int32),
                ("history_bf16", ctypes.c_int32), ("gram_fusion", ctypes.c_int32), ("ritz_columns", ctypes.c_int32),
                ("moments_bf16", ctypes.c_int32), ("small_rank_path", ctypes.c_int32)]


_vp = ctypes.c_void_p
_lib.ngalore_create.restype = ctypes.c_int
_lib.ngalore_create.argtypes = [ctypes.POINTER(Shape), ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                ctypes.c_double, ctypes.c_double, ctypes.c_double, ctypes.c_double,
                                ctypes.c_double, ctypes.c_double, ctypes.POINTER(Options), ctypes.POINTER(_vp)]
_lib.ngalore_destroy.restype = None
_lib.ngalore_destroy.argtypes = [_vp]
_lib.ngalore_step.restype = ctypes.c_int
_lib.ngalore_step.argtypes = [_vp, ctypes.POINTER(_vp), ctypes.POINTER(_vp), _vp]
_lib.ngalore_refresh_subspace.restype = ctypes.c_int
_lib.ngalore_refresh_subspace.argtypes = [_vp, ctypes.POINTER(_vp), ctypes.c_int, _vp]
_lib.ngalore_step_host.restype = ctypes.c_int
_lib.ngalore_step_host.argtypes = [_vp, ctypes.POINTER(_vp), ctypes.POINTER(_vp), _vp]
_lib.ngalore_poll_status.restype = ctypes.c_int
_lib.ngalore_poll_status.argtypes = [_vp, ctypes.POINTER(ctypes.c_int)]
for _name in ("ngalore_get_subspace", "ngalore_set_subspace", "ngalore_get_working_subspace"):
    getattr(_lib, _name).restype = ctypes.c_int
    getattr(_lib, _name).argtypes = [_vp, ctypes.c_int, _vp, _vp]
_lib.ngalore_state_export.restype = ctypes.c_int
_lib.ngalore_state_export.argtypes = [_vp, _vp, ctypes.POINTER(ctypes.c_size_t)]
_lib.ngalore_state_import.restype = ctypes.c_int
_lib.ngalore_state_import.argtypes = [_vp, _vp, ctypes.c_size_t]
_lib.ngalore_set_update_groups.restype = ctypes.c_int
_lib.ngalore_set_update_groups.argtypes = [_vp, ctypes.c_int]
_lib.ngalore_num_update_groups.restype = ctypes.c_int
_lib.ngalore_num_update_groups.argtypes = [_vp]
_lib.ngalore_update_group_range.restype = ctypes.c_int
_lib.ngalore_update_group_range.argtypes = [_vp, ctypes.c_int, ctypes.POINTER(ctypes.c_int), ctypes.POINTER(ctypes.c_int)]
_lib.ngalore_stream_wait_update.restype = ctypes.c_int
_lib.ngalore_stream_wait_update.argtypes = [_vp, ctypes.c_int, _vp]
_lib.ngalore_debug_withhold_solution.restype = ctypes.c_int
_lib.ngalore_debug_withhold_solution.argtypes = [_vp, ctypes.c_int, ctypes.c_int]
_lib.ngalore_set_lr.restype = ctypes.c_int
_lib.ngalore_set_lr.argtypes = [_vp, ctypes.c_double]
_lib.ngalore_num_matrices.restype = ctypes.c_int
_lib.ngalore_num_matrices.argtypes = [_vp]
for _name in ("ngalore_rank", "ngalore_projects_right", "ngalore_subspace_rows"):
    getattr(_lib, _name).restype = ctypes.c_int
    getattr(_lib, _name).argtypes = [_vp, ctypes.c_int]
_lib.ngalore_step_count.restype = ctypes.c_int64
_lib.ngalore_step_count.argtypes = [_vp]
_lib.ngalore_device_bytes.restype = ctypes.c_size_t
_lib.ngalore_device_bytes.argtypes = [_vp]
_lib.ngalore_launch_count.restype = ctypes.c_int64
_lib.ngalore_launch_count.argtypes = [_vp]
_lib.ngalore_uses_small_rank_path.restype = ctypes.c_int
_lib.ngalore_uses_small_rank_path.argtypes = [_vp]
_lib.ngalore_descriptor_uploads.restype = ctypes.c_int64
_lib.ngalore_descriptor_uploads.argtypes = [_vp]
_lib.ngalore_set_profiling.restype = ctypes.c_int
_lib.ngalore_set_profiling.argtypes = [_vp, ctypes.c_int]
_lib.ngalore_last_phase_ms.restype = ctypes.c_double
_lib.ngalore_last_phase_ms.argtypes = [_vp, ctypes.c_int]
_lib.ngalore_natural_gradient_static.restype = ctypes.c_int
_lib.ngalore_natural_gradient_static.argtypes = [_vp, ctypes.c_int64, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                                 ctypes.c_double, _vp, _vp, _vp, _vp]
_lib.ngalore_status_string.restype = ctypes.c_char_p
_lib.ngalore_status_string.argtypes = [ctypes.c_int]


class NGaLoreError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {STATUS_NAMES.get(code, code)} ({_lib.ngalore_status_string(code).decode()})")


def _check(code: int, where: str) -> None:
    if code != OK:
        raise NGaLoreError(code, where)


def _stream_ptr(stream) -> Optional[int]:
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def _ptr_array(tensors: Sequence[torch.Tensor]):
    arr = (_vp * len(tensors))()
    for i, t in enumerate(tensors):
        arr[i] = t.data_ptr()
    return arr


class NGaLore:
    """Optimizer state for a list of (rows, cols) weight matrices on the current CUDA device."""

    def __init__(self, shapes, r, s, T, lam=1e-3, lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, wd=0.0, *,
                 gemm_impl=0, stream_impl=0, power_iterations=0, reset_history_on_refresh=False, seed=0,
                 projection="left", history_bf16=False, gram_fusion=False, ritz_columns=0,
                 moments_bf16=False, small_rank_path=False):
        self.shapes = [(int(M), int(N)) for M, N in shapes]
        arr = (Shape * len(self.shapes))(*[Shape(M, N) for M, N in self.shapes])
        rule = {"left": 0, "short_side": 1}[projection]
        opt = Options(ctypes.sizeof(Options), gemm_impl, power_iterations, int(reset_history_on_refresh), seed,
                      stream_impl, rule, int(history_bf16), 1 if gram_fusion else 0, ritz_columns,
                      int(moments_bf16), 1 if small_rank_path else 0)
        handle = _vp()
        _check(_lib.ngalore_create(arr, len(self.shapes), r, s, T, lam, lr, beta1, beta2, eps, wd,
                                   ctypes.byref(opt), ctypes.byref(handle)), "ngalore_create")
        self._h = handle
        self.device = torch.device("cuda", torch.cuda.current_device())

    def close(self):
        if getattr(self, "_h", None):
            _lib.ngalore_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- checks ---------------------------------------------------------------
    def _check_WG(self, W, G):
        assert len(W) == len(self.shapes) and len(G) == len(self.shapes)
        for (M, N), w, g in zip(self.shapes, W, G):
            assert w.is_cuda and w.dtype == torch.float32 and w.is_contiguous() and tuple(w.shape) == (M, N)
            assert g.is_cuda and g.dtype == torch.bfloat16 and g.is_contiguous() and tuple(g.shape) == (M, N)

    # -- the three calls of the optimizer -------------------------------------------
    def step(self, W: List[torch.Tensor], G: List[torch.Tensor], stream=None, check=True):
        if check:
            self._check_WG(W, G)
        _check(_lib.ngalore_step(self._h, _ptr_array(W), _ptr_array(G), _stream_ptr(stream)), "ngalore_step")

    def step_ptrs(self, W_ptrs, G_ptrs, stream=None):
        """Step with pre-built pointer arrays (see ``pointer_array``): no per-call marshalling."""
        _check(_lib.ngalore_step(self._h, W_ptrs, G_ptrs, _stream_ptr(stream)), "ngalore_step")

    @staticmethod
    def pointer_array(tensors):
        return _ptr_array(tensors)

    def refresh_subspace(self, G: List[torch.Tensor], matrix_index=-1, stream=None):
        assert len(G) == len(self.shapes)
        _check(_lib.ngalore_refresh_subspace(self._h, _ptr_array(G), matrix_index, _stream_ptr(stream)),
               "ngalore_refresh_subspace")

    def step_host(self, W_host: List[torch.Tensor], G_host: List[torch.Tensor], stream=None):
        """Step with host tensors (fp32 W updated in place, bf16 G); copies run inside the call."""
        for w, g in zip(W_host, G_host):
            assert not w.is_cuda and not g.is_cuda and w.is_contiguous() and g.is_contiguous()
        _check(_lib.ngalore_step_host(self._h, _ptr_array(W_host), _ptr_array(G_host), _stream_ptr(stream)),
               "ngalore_step_host")

    # -- state access -----------------------------------------------------------
    def poll_status(self):
        arr = (ctypes.c_int * len(self.shapes))()
        code = _lib.ngalore_poll_status(self._h, arr)
        return code, list(arr)

    def rank(self, i):
        return _lib.ngalore_rank(self._h, i)

    def projects_right(self, i) -> bool:
        return _lib.ngalore_projects_right(self._h, i) == 1

    def subspace_rows(self, i):
        return _lib.ngalore_subspace_rows(self._h, i)

    def get_subspace(self, i, working=False) -> torch.Tensor:
        out = torch.empty((self.subspace_rows(i), self.rank(i)), dtype=torch.float32, device=self.device)
        fn = _lib.ngalore_get_working_subspace if working else _lib.ngalore_get_subspace
        _check(fn(self._h, i, out.data_ptr(), _stream_ptr(None)), "ngalore_get_subspace")
        return out

    def set_subspace(self, i, P: torch.Tensor):
        P = P.to(device=self.device, dtype=torch.float32).contiguous()
        assert tuple(P.shape) == (self.subspace_rows(i), self.rank(i))
        _check(_lib.ngalore_set_subspace(self._h, i, P.data_ptr(), _stream_ptr(None)), "ngalore_set_subspace")
        torch.cuda.current_stream().synchronize()  # P may be freed by the caller

    def export_state(self) -> bytes:
        n = ctypes.c_size_t(0)
        _check(_lib.ngalore_state_export(self._h, None, ctypes.byref(n)), "ngalore_state_export")
        buf = ctypes.create_string_buffer(n.value)
        _check(_lib.ngalore_state_export(self._h, buf, ctypes.byref(n)), "ngalore_state_export")
        return buf.raw[: n.value]

    def import_state(self, blob: bytes):
        _check(_lib.ngalore_state_import(self._h, blob, len(blob)), "ngalore_state_import")

    def set_update_groups(self, n_groups: int):
        """Run the weight update in n_groups launches with an event after each (see include/ngalore.h)."""
        _check(_lib.ngalore_set_update_groups(self._h, n_groups), "ngalore_set_update_groups")

    def update_groups(self):
        """[(first, last), ...]: the matrix ranges of the update groups (one range when groups are off)."""
        out = []
        for g in range(_lib.ngalore_num_update_groups(self._h)):
            a, b = ctypes.c_int(0), ctypes.c_int(0)
            _check(_lib.ngalore_update_group_range(self._h, g, ctypes.byref(a), ctypes.byref(b)), "ngalore_update_group_range")
            out.append((a.value, b.value))
        return out

    def stream_wait_update(self, g: int, stream):
        """Make `stream` (a torch.cuda.Stream) wait until the latest enqueued step has updated group g."""
        _check(_lib.ngalore_stream_wait_update(self._h, g, ctypes.c_void_p(stream.cuda_stream)), "ngalore_stream_wait_update")

    def debug_withhold_solution(self, matrix_index: int, polls: int):
        """Testing aid: the next step does not announce matrix_index's solved weights (see include/ngalore.h)."""
        _check(_lib.ngalore_debug_withhold_solution(self._h, matrix_index, polls), "ngalore_debug_withhold_solution")

    def set_lr(self, lr: float):
        _check(_lib.ngalore_set_lr(self._h, lr), "ngalore_set_lr")

    @property
    def step_count(self) -> int:
        return _lib.ngalore_step_count(self._h)

    @property
    def device_bytes(self) -> int:
        return _lib.ngalore_device_bytes(self._h)

    @property
    def launch_count(self) -> int:
        return _lib.ngalore_launch_count(self._h)

    @property
    def uses_small_rank_path(self) -> bool:
        return _lib.ngalore_uses_small_rank_path(self._h) == 1

    @property
    def descriptor_uploads(self) -> int:
        return _lib.ngalore_descriptor_uploads(self._h)

    def set_profiling(self, on: bool):
        _check(_lib.ngalore_set_profiling(self._h, int(on)), "ngalore_set_profiling")

    def last_phase_ms(self, phase: int) -> float:
        return _lib.ngalore_last_phase_ms(self._h, phase)


def natural_gradient_static(H: torch.Tensor, count: int, cur: int, lam: float, K: torch.Tensor, out: torch.Tensor,
                            status: Optional[torch.Tensor] = None, stream=None) -> None:
    """Allocation-free natural-gradient transform (ngalore_natural_gradient_static).

    H: (s, n) fp32 history ring on the device, K: (s, s) fp64 raw Gram matrix kept by the caller
    (zeros before the first call), out: (n,) fp32.  For callers that may not allocate device memory:
    the library's scratch is a fixed array inside the library image (n <= 8,388,608).  Calls share
    that array, so keep them on one stream."""
    assert H.is_cuda and H.dtype == torch.float32 and H.is_contiguous() and H.dim() == 2
    assert K.is_cuda and K.dtype == torch.float64 and K.is_contiguous() and tuple(K.shape) == (H.shape[0],) * 2
    assert out.is_cuda and out.dtype == torch.float32 and out.is_contiguous() and out.numel() == H.shape[1]
    sp = status.data_ptr() if status is not None else None
    _check(_lib.ngalore_natural_gradient_static(H.data_ptr(), H.shape[1], H.shape[0], count, cur, lam, K.data_ptr(),
                                                out.data_ptr(), sp, _stream_ptr(stream)),
           "ngalore_natural_gradient_static")
