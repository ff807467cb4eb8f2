"""ctypes binding of libbra_b200.so: same names as the C boundary (include/bra.h).

Argument marshalling only.  PyTorch provides device memory and the CUDA
stream; every step of the path runs inside the library's kernels.  If the
library has not been built, or there is no CUDA device, calls raise: there is
no fallback.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import c_float, c_int32, c_size_t, c_void_p

_LIB = None
_LIB_NAME = "libbra_b200.so"

IMPL_AUTO, IMPL_SIMT, IMPL_MMA, IMPL_TC, IMPL_IMG, IMPL_TC_FUSED = 0, 1, 2, 3, 4, 5
F32, BF16 = 0, 1


class BraProblem(ctypes.Structure):
    """Mirror of `bra_problem` (Algorithm 1 notation: H, W, C, S, k, plus batch and heads)."""

    _fields_ = [
        ("B", c_int32), ("H", c_int32), ("W", c_int32), ("C", c_int32),
        ("heads", c_int32), ("S", c_int32), ("topk", c_int32), ("dtype", c_int32),
        ("scale", c_float), ("shared_routing", c_int32), ("lce_ksize", c_int32), ("impl", c_int32),
        ("inject", c_int32),
    ]

    @property
    def R(self):
        return self.S * self.S

    @property
    def heads_i(self):
        return 1 if self.shared_routing else self.heads


class BraError(RuntimeError):
    def __init__(self, code, where):
        self.code = int(code)
        super().__init__(f"{where}: {status_string(code)} (bra_status {int(code)})")


def library_path() -> str:
    """The built library next to this file, or the file BRA_LIBRARY_PATH names (to try another build)."""
    return os.environ.get("BRA_LIBRARY_PATH") or os.path.join(os.path.dirname(os.path.abspath(__file__)), _LIB_NAME)


def load_library():
    """Load the built library (never builds it; see build.py / __graft_entry__.build)."""
    global _LIB
    if _LIB is not None:
        return _LIB
    path = library_path()
    if not os.path.exists(path):
        raise RuntimeError(
            f"{path} is missing: build it with `python -m paper_2303_08810_b200.build` "
            "(there is no CPU fallback)")
    lib = ctypes.CDLL(path)
    P = ctypes.POINTER(BraProblem)
    v = c_void_p
    lib.bra_workspace_bytes.restype = c_size_t
    lib.bra_workspace_bytes.argtypes = [P]
    lib.bra_workspace_init.restype = c_int32
    lib.bra_workspace_init.argtypes = [P, v, c_size_t, v]
    lib.bra_route.restype = c_int32
    lib.bra_route.argtypes = [P, v, v, v, v, v, v, c_size_t, v]
    lib.bra_route_static.restype = c_int32
    lib.bra_route_static.argtypes = [P, v, v, v, v]
    lib.bra_attend.restype = c_int32
    lib.bra_attend.argtypes = [P, v, v, v, v, v, v, v, v, v, c_size_t, v]
    lib.bra_forward.restype = c_int32
    lib.bra_forward.argtypes = [P, v, v, v, v, v, v, v, v, v, c_size_t, v]
    lib.bra_backward.restype = c_int32
    lib.bra_backward.argtypes = [P] + [v] * 12 + [v, c_size_t, v]
    lib.bra_device_status.restype = c_int32
    lib.bra_device_status.argtypes = [v, v]
    lib.bra_last_launch_count.restype = c_int32
    lib.bra_last_launch_count.argtypes = []
    lib.bra_status_string.restype = ctypes.c_char_p
    lib.bra_status_string.argtypes = [c_int32]
    lib.bra_version.restype = c_int32
    lib.bra_version.argtypes = []
    _LIB = lib
    return lib


def status_string(code) -> str:
    return load_library().bra_status_string(int(code)).decode()


def version() -> int:
    return load_library().bra_version()


def last_launch_count() -> int:
    return load_library().bra_last_launch_count()


def make_problem(B, H, W, C, heads, S, topk, dtype="bf16", scale=0.0, shared_routing=False,
                 lce=True, impl=IMPL_AUTO, inject=0) -> BraProblem:
    dt = {"f32": F32, "bf16": BF16, F32: F32, BF16: BF16}[dtype]
    return BraProblem(B, H, W, C, heads, S, topk, dt, float(scale), int(bool(shared_routing)),
                      5 if lce else 0, int(impl), int(inject))


def workspace_bytes(p: BraProblem) -> int:
    return int(load_library().bra_workspace_bytes(ctypes.byref(p)))


def _torch():
    import torch
    if not torch.cuda.is_available():
        raise RuntimeError("paper_2303_08810_b200 needs a CUDA device (no CPU fallback)")
    return torch


def workspace(p: BraProblem, device="cuda"):
    """Zero-filled scratch tensor of bra_workspace_bytes(p) bytes."""
    torch = _torch()
    n = workspace_bytes(p)
    if n == 0:
        raise BraError(2, "bra_workspace_bytes")
    return torch.zeros(n, dtype=torch.uint8, device=device)


def workspace_init(p: BraProblem, ws, stream=None):
    """bra_workspace_init: status block, job counters and flags of `ws` set to zero."""
    _check(load_library().bra_workspace_init(ctypes.byref(p), _ptr(ws), ws.numel(), _stream(stream)),
           "bra_workspace_init")
    return ws


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _stream(stream):
    if stream is None:
        return _torch().cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def _tdtype(p):
    torch = _torch()
    return torch.bfloat16 if p.dtype == BF16 else torch.float32


def _check(code, where):
    if code != 0:
        raise BraError(code, where)


def bra_route(p, Q, K, q_mean=None, k_mean=None, index=None, ws=None, stream=None, want_means=True):
    """bra_route: Q, K -> (q_mean, k_mean, index)."""
    torch = _torch()
    lib = load_library()
    ws = workspace(p, Q.device) if ws is None else ws
    if want_means:
        q_mean = torch.empty(p.B, p.R, p.C, dtype=torch.float32, device=Q.device) if q_mean is None else q_mean
        k_mean = torch.empty(p.B, p.R, p.C, dtype=torch.float32, device=Q.device) if k_mean is None else k_mean
    if index is None:
        index = torch.empty(p.B, p.heads_i, p.R, p.topk, dtype=torch.int32, device=Q.device)
    _check(lib.bra_route(ctypes.byref(p), _ptr(Q), _ptr(K), _ptr(q_mean), _ptr(k_mean), _ptr(index),
                         _ptr(ws), ws.numel(), _stream(stream)), "bra_route")
    return q_mean, k_mean, index


ROUTE_STATIC_MAX_MEAN_FLOATS = 512 * 1024


def bra_route_static(p, Q, K, index=None, stream=None):
    """bra_route_static: Q, K -> index, for callers that have no scratch buffer to give.

    The region means stay inside the library (a fixed array of
    2 x ROUTE_STATIC_MAX_MEAN_FLOATS floats per GPU); the C call allocates
    nothing.  Pass a preallocated `index` to keep the whole call allocation-free:
    only when `index` is None does this wrapper ask torch for one.  Calls on
    one device share the array, so keep them ordered on a stream.
    """
    torch = _torch()
    lib = load_library()
    if index is None:
        index = torch.empty(p.B, p.heads_i, p.R, p.topk, dtype=torch.int32, device=Q.device)
    _check(lib.bra_route_static(ctypes.byref(p), _ptr(Q), _ptr(K), _ptr(index), _stream(stream)),
           "bra_route_static")
    return index


def bra_attend(p, Q, K, V, index, lce_w=None, lce_b=None, O=None, lse=None, ws=None, stream=None,
               want_lse=True):
    """bra_attend: Q, K, V, index -> (O, lse)."""
    torch = _torch()
    lib = load_library()
    ws = workspace(p, Q.device) if ws is None else ws
    O = torch.empty_like(Q) if O is None else O
    if lse is None and want_lse:
        lse = torch.empty(p.B, p.heads, p.H * p.W, dtype=torch.float32, device=Q.device)
    _check(lib.bra_attend(ctypes.byref(p), _ptr(Q), _ptr(K), _ptr(V), _ptr(index), _ptr(lce_w),
                          _ptr(lce_b), _ptr(O), _ptr(lse), _ptr(ws), ws.numel(), _stream(stream)),
           "bra_attend")
    return O, lse


def bra_forward(p, Q, K, V, lce_w=None, lce_b=None, O=None, index=None, lse=None, ws=None,
                stream=None, want_index=True, want_lse=True):
    """bra_forward: Q, K, V -> (O, index, lse)."""
    torch = _torch()
    lib = load_library()
    ws = workspace(p, Q.device) if ws is None else ws
    O = torch.empty_like(Q) if O is None else O
    if index is None and want_index:
        index = torch.empty(p.B, p.heads_i, p.R, p.topk, dtype=torch.int32, device=Q.device)
    if lse is None and want_lse:
        lse = torch.empty(p.B, p.heads, p.H * p.W, dtype=torch.float32, device=Q.device)
    _check(lib.bra_forward(ctypes.byref(p), _ptr(Q), _ptr(K), _ptr(V), _ptr(lce_w), _ptr(lce_b),
                           _ptr(O), _ptr(index), _ptr(lse), _ptr(ws), ws.numel(), _stream(stream)),
           "bra_forward")
    return O, index, lse


def bra_backward(p, Q, K, V, index, lce_w, lse, dO, dQ=None, dK=None, dV=None, d_lce_w=None,
                 d_lce_b=None, ws=None, stream=None, want_bias_grad=False):
    """bra_backward: -> (dQ, dK, dV, d_lce_w, d_lce_b)."""
    torch = _torch()
    lib = load_library()
    ws = workspace(p, Q.device) if ws is None else ws
    dQ = torch.empty_like(Q) if dQ is None else dQ
    dK = torch.empty_like(K) if dK is None else dK
    dV = torch.empty_like(V) if dV is None else dV
    if d_lce_w is None and p.lce_ksize:
        d_lce_w = torch.empty(p.C, 5, 5, dtype=torch.float32, device=Q.device)
    if d_lce_b is None and want_bias_grad:
        d_lce_b = torch.empty(p.C, dtype=torch.float32, device=Q.device)
    _check(lib.bra_backward(ctypes.byref(p), _ptr(Q), _ptr(K), _ptr(V), _ptr(index), _ptr(lce_w),
                            _ptr(lse), _ptr(dO), _ptr(dQ), _ptr(dK), _ptr(dV), _ptr(d_lce_w),
                            _ptr(d_lce_b), _ptr(ws), ws.numel(), _stream(stream)), "bra_backward")
    return dQ, dK, dV, d_lce_w, d_lce_b


def bra_device_status(ws, stream=None) -> int:
    """Synchronise the stream and return (and clear) the first device-detected error in ws."""
    return int(load_library().bra_device_status(_ptr(ws), _stream(stream)))
