"""Thin ctypes binding over libgptq2d.so (the C ABI of include/gptq2d.h).

Argument marshalling only: every step of the method runs in the CUDA library.
PyTorch supplies device memory and streams.  There is no CPU fallback: importing
this module raises if the library has not been built.

Function names mirror the C entry points.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# GPTQ2D_LIBRARY selects another build of the same library (the tests use it for the checked build,
# libgptq2d_checked.so, in a process of its own); it must name a file inside this package
_LIB_PATH = os.path.join(_HERE, os.path.basename(os.environ.get("GPTQ2D_LIBRARY", "libgptq2d.so")))

FP64, FP32, FP64_UNTILED, FP64_PULL, FP32_UNTILED = 0, 1, 2, 3, 4

OK = 0
STATUS_NAMES = {
    0: "OK", 1: "ERR_INVALID_ARG", 2: "ERR_WORKSPACE", 3: "ERR_UNSUPPORTED_DEVICE", 4: "ERR_CUDA",
    5: "ERR_NOT_SPD", 6: "ERR_NONFINITE", 7: "ERR_INT_OVERFLOW", 8: "ERR_DEVICE_TIMEOUT",
    9: "ERR_TOO_LARGE", 10: "ERR_CHECK",
}

EXPORTS = (
    "gptq2d_status_string", "gptq2d_factor_workspace_bytes", "gptq2d_factor",
    "gptq2d_round_workspace_bytes", "gptq2d_round", "gptq2d_round_host_workspace_bytes",
    "gptq2d_round_host", "gptq2d_objective_workspace_bytes", "gptq2d_objective",
    "gptq2d_round_static", "gptq2d_round_static_max_dim",
    "gptq2d_round_batched_workspace_bytes", "gptq2d_round_batched",
    "gptq2d_factor_reverse_workspace_bytes", "gptq2d_factor_reverse",
    "gptq2d_round_reverse_workspace_bytes", "gptq2d_round_reverse",
    "gptq2d_round_f32in_workspace_bytes", "gptq2d_round_f32in",
    "gptq2d_round_blocked_workspace_bytes", "gptq2d_round_blocked",
    "gptq2d_factor_batched_workspace_bytes", "gptq2d_factor_batched",
    "gptq2d_internal_test_hook", "gptq2d_internal_gemm",
)
FACTOR_SMALL_MAX = 128

BLOCKED_MAX_WIDTH = 64

BATCH_MAX_COUNT, BATCH_MAX_DIM = 8192, 32768


class Problem(ctypes.Structure):
    """gptq2d_problem_t: one matrix of a batched sweep (device pointers, leading dimensions in elements)."""
    _fields_ = [("m", ctypes.c_int), ("n", ctypes.c_int),
                ("X", ctypes.c_void_p), ("ldx", ctypes.c_long),
                ("L", ctypes.c_void_p), ("ldl", ctypes.c_long),
                ("U", ctypes.c_void_p), ("ldu", ctypes.c_long),
                ("Z", ctypes.c_void_p), ("ldz", ctypes.c_long),
                ("E", ctypes.c_void_p), ("lde", ctypes.c_long)]


class FactorProblem(ctypes.Structure):
    """gptq2d_factor_problem_t: one (A, B) pair of a batched set-up (device pointers; A or B may be NULL)."""
    _fields_ = [("m", ctypes.c_int), ("n", ctypes.c_int),
                ("A", ctypes.c_void_p), ("lda", ctypes.c_long),
                ("B", ctypes.c_void_p), ("ldb", ctypes.c_long),
                ("L", ctypes.c_void_p), ("ldl", ctypes.c_long),
                ("U", ctypes.c_void_p), ("ldu", ctypes.c_long),
                ("dL", ctypes.c_void_p), ("dU", ctypes.c_void_p)]


class Gptq2dError(RuntimeError):
    def __init__(self, status, info=None):
        self.status = int(status)
        self.info = info
        name = STATUS_NAMES.get(self.status, str(status))
        super().__init__("gptq2d: %s%s" % (name, "" if info is None else " info=%s" % (list(info),)))


def _load():
    if not os.path.exists(_LIB_PATH):
        raise ImportError(
            "libgptq2d.so is not built (%s). Run `python -m paper_2607_27042_b200.build` "
            "or __graft_entry__.build(); there is no CPU fallback." % _LIB_PATH)
    lib = ctypes.CDLL(_LIB_PATH)
    c = ctypes
    vp, sz, i32, lng = c.c_void_p, c.c_size_t, c.c_int, c.c_long
    lib.gptq2d_status_string.restype = c.c_char_p
    lib.gptq2d_status_string.argtypes = [i32]
    for name in ("gptq2d_factor_workspace_bytes", "gptq2d_objective_workspace_bytes"):
        getattr(lib, name).restype = sz
        getattr(lib, name).argtypes = [i32, i32]
    for name in ("gptq2d_round_workspace_bytes", "gptq2d_round_host_workspace_bytes"):
        getattr(lib, name).restype = sz
        getattr(lib, name).argtypes = [i32, i32, i32]
    lib.gptq2d_factor.restype = i32
    lib.gptq2d_factor.argtypes = [i32, i32, vp, lng, vp, lng, vp, lng, vp, lng, vp, vp, vp, sz, vp, vp]
    lib.gptq2d_round.restype = i32
    lib.gptq2d_round.argtypes = [i32, i32, vp, lng, vp, lng, vp, lng, vp, lng, vp, lng, vp, i32, vp, sz, vp, vp]
    lib.gptq2d_round_host.restype = i32
    lib.gptq2d_round_host.argtypes = [i32, i32, vp, vp, vp, vp, vp, vp, i32, vp, sz, vp, vp]
    lib.gptq2d_objective.restype = i32
    lib.gptq2d_objective.argtypes = [i32, i32, vp, lng, vp, lng, vp, lng, vp, lng, vp, vp, sz, vp, vp]
    lib.gptq2d_round_static.restype = i32
    lib.gptq2d_round_static.argtypes = [i32, i32, vp, lng, vp, lng, vp, lng, vp, lng, vp, lng, vp, vp, vp]
    lib.gptq2d_internal_gemm.restype = i32
    lib.gptq2d_internal_gemm.argtypes = [i32, i32, i32, i32, i32, c.c_double, vp, lng, vp, lng, c.c_double, vp, lng, vp]
    lib.gptq2d_internal_test_hook.restype = i32
    lib.gptq2d_internal_test_hook.argtypes = [i32, lng]
    lib.gptq2d_round_static_max_dim.restype = sz
    lib.gptq2d_round_static_max_dim.argtypes = []
    lib.gptq2d_round_f32in.restype = i32
    lib.gptq2d_round_f32in.argtypes = [i32, i32, vp, lng, vp, lng, vp, lng, vp, lng, vp, lng, vp, vp, sz, vp, vp]
    lib.gptq2d_factor_batched_workspace_bytes.restype = sz
    lib.gptq2d_factor_batched_workspace_bytes.argtypes = [i32, vp]
    lib.gptq2d_factor_batched.restype = i32
    lib.gptq2d_factor_batched.argtypes = [i32, vp, vp, sz, vp, vp]
    lib.gptq2d_round_blocked_workspace_bytes.restype = sz
    lib.gptq2d_round_blocked_workspace_bytes.argtypes = [i32, i32, i32]
    lib.gptq2d_round_blocked.restype = i32
    lib.gptq2d_round_blocked.argtypes = [i32, i32, vp, lng, vp, lng, vp, lng, i32, vp, lng, vp, lng, vp, vp, sz, vp, vp]
    for name in ("gptq2d_factor_reverse_workspace_bytes", "gptq2d_round_reverse_workspace_bytes",
                 "gptq2d_round_f32in_workspace_bytes"):
        getattr(lib, name).restype = sz
        getattr(lib, name).argtypes = [i32, i32]
    lib.gptq2d_factor_reverse.restype = i32
    lib.gptq2d_factor_reverse.argtypes = [i32, i32, vp, lng, vp, lng, vp, lng, vp, lng, vp, vp, vp, sz, vp, vp]
    lib.gptq2d_round_reverse.restype = i32
    lib.gptq2d_round_reverse.argtypes = [i32, i32, vp, lng, vp, lng, vp, lng, vp, lng, vp, lng, vp, vp, sz, vp, vp]
    lib.gptq2d_round_batched_workspace_bytes.restype = sz
    lib.gptq2d_round_batched_workspace_bytes.argtypes = [i32, vp]
    lib.gptq2d_round_batched.restype = i32
    lib.gptq2d_round_batched.argtypes = [i32, vp, vp, vp, sz, vp, vp]
    return lib


_lib = _load()


def library_path():
    return _LIB_PATH


def status_string(status):
    return _lib.gptq2d_status_string(int(status)).decode()


def _stream_ptr(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def _mat(t, dtype, name):
    if t is None:
        return None, 0
    if not (t.is_cuda and t.dtype == dtype and t.dim() == 2 and t.stride(1) == 1):
        raise ValueError("%s must be a 2-D CUDA tensor of %s with unit column stride" % (name, dtype))
    return ctypes.c_void_p(t.data_ptr()), int(t.stride(0))


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _workspace(nbytes, device):
    # torch's caching allocator returns 512-byte aligned blocks
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)


def check_info(info):
    """Synchronises and raises if the device reported a data-dependent error."""
    vals = info.cpu().tolist()
    if vals[0] != 0:
        raise Gptq2dError(vals[0], vals)


def gptq2d_factor_workspace_bytes(m, n):
    return int(_lib.gptq2d_factor_workspace_bytes(m, n))


def gptq2d_round_workspace_bytes(m, n, precision=FP64):
    return int(_lib.gptq2d_round_workspace_bytes(m, n, precision))


def gptq2d_round_host_workspace_bytes(m, n, precision=FP64):
    return int(_lib.gptq2d_round_host_workspace_bytes(m, n, precision))


def gptq2d_objective_workspace_bytes(m, n):
    return int(_lib.gptq2d_objective_workspace_bytes(m, n))


def gptq2d_factor(A, B, L=None, U=None, dL=None, dU=None, workspace=None, info=None, stream=None, m=None, n=None):
    """L, U (and 1/Lambda_L, 1/Lambda_U) from the bases A (m x m) and B (n x n).

    A or B may be None (identity) if m / n is given.  Returns (L, U, dL, dU, info)."""
    m = A.shape[0] if A is not None else m
    n = B.shape[0] if B is not None else n
    dev = (A if A is not None else B).device if (A is not None or B is not None) else torch.device("cuda")
    L = torch.empty((m, m), dtype=torch.float64, device=dev) if L is None else L
    U = torch.empty((n, n), dtype=torch.float64, device=dev) if U is None else U
    dL = torch.empty(m, dtype=torch.float64, device=dev) if dL is None else dL
    dU = torch.empty(n, dtype=torch.float64, device=dev) if dU is None else dU
    info = torch.zeros(4, dtype=torch.int32, device=dev) if info is None else info
    nbytes = gptq2d_factor_workspace_bytes(m, n)
    workspace = _workspace(nbytes, dev) if workspace is None else workspace
    pA, lda = _mat(A, torch.float64, "A")
    pB, ldb = _mat(B, torch.float64, "B")
    pL, ldl = _mat(L, torch.float64, "L")
    pU, ldu = _mat(U, torch.float64, "U")
    st = _lib.gptq2d_factor(m, n, pA, lda, pB, ldb, pL, ldl, pU, ldu, _ptr(dL), _ptr(dU),
                            _ptr(workspace), workspace.numel(), _ptr(info), _stream_ptr(stream))
    if st != OK:
        raise Gptq2dError(st)
    return L, U, dL, dU, info


def gptq2d_round(X, L, U, Z=None, E=None, min_margin=None, precision=FP64, workspace=None, info=None,
                 stream=None, want_E=False, want_margin=False):
    """The sweep.  Returns (Z, E, min_margin, info); E / min_margin are None unless asked for."""
    m, n = X.shape
    dev = X.device
    Z = torch.empty((m, n), dtype=torch.int32, device=dev) if Z is None else Z
    if E is None and want_E:
        E = torch.empty((m, n), dtype=torch.float64, device=dev)
    if min_margin is None and want_margin:
        min_margin = torch.empty(1, dtype=torch.float64, device=dev)
    info = torch.zeros(4, dtype=torch.int32, device=dev) if info is None else info
    nbytes = gptq2d_round_workspace_bytes(m, n, precision)
    workspace = _workspace(nbytes, dev) if workspace is None else workspace
    pX, ldx = _mat(X, torch.float64, "X")
    pL, ldl = _mat(L, torch.float64, "L")
    pU, ldu = _mat(U, torch.float64, "U")
    pZ, ldz = _mat(Z, torch.int32, "Z")
    pE, lde = _mat(E, torch.float64, "E")
    st = _lib.gptq2d_round(m, n, pX, ldx, pL, ldl, pU, ldu, pZ, ldz, pE, lde, _ptr(min_margin), int(precision),
                           _ptr(workspace), workspace.numel(), _ptr(info), _stream_ptr(stream))
    if st != OK:
        raise Gptq2dError(st)
    return Z, E, min_margin, info


def gptq2d_factor_reverse_workspace_bytes(m, n):
    return int(_lib.gptq2d_factor_reverse_workspace_bytes(m, n))


def gptq2d_round_reverse_workspace_bytes(m, n):
    return int(_lib.gptq2d_round_reverse_workspace_bytes(m, n))


def gptq2d_factor_reverse(A, B, Lr=None, Ur=None, dL=None, dU=None, workspace=None, info=None, stream=None,
                          m=None, n=None):
    """Factors for the reverse order: Lr unit upper, Ur unit lower.  Returns (Lr, Ur, dL, dU, info)."""
    m = A.shape[0] if A is not None else m
    n = B.shape[0] if B is not None else n
    dev = (A if A is not None else B).device if (A is not None or B is not None) else torch.device("cuda")
    Lr = torch.empty((m, m), dtype=torch.float64, device=dev) if Lr is None else Lr
    Ur = torch.empty((n, n), dtype=torch.float64, device=dev) if Ur is None else Ur
    dL = torch.empty(m, dtype=torch.float64, device=dev) if dL is None else dL
    dU = torch.empty(n, dtype=torch.float64, device=dev) if dU is None else dU
    info = torch.zeros(4, dtype=torch.int32, device=dev) if info is None else info
    workspace = _workspace(gptq2d_factor_reverse_workspace_bytes(m, n), dev) if workspace is None else workspace
    pA, lda = _mat(A, torch.float64, "A")
    pB, ldb = _mat(B, torch.float64, "B")
    pL, ldl = _mat(Lr, torch.float64, "Lr")
    pU, ldu = _mat(Ur, torch.float64, "Ur")
    st = _lib.gptq2d_factor_reverse(m, n, pA, lda, pB, ldb, pL, ldl, pU, ldu, _ptr(dL), _ptr(dU),
                                    _ptr(workspace), workspace.numel(), _ptr(info), _stream_ptr(stream))
    if st != OK:
        raise Gptq2dError(st)
    return Lr, Ur, dL, dU, info


def gptq2d_round_reverse(X, Lr, Ur, Z=None, E=None, min_margin=None, workspace=None, info=None, stream=None,
                         want_E=False, want_margin=False):
    """The sweep in reverse order (from the last row and column).  Returns (Z, E, min_margin, info)."""
    m, n = X.shape
    dev = X.device
    Z = torch.empty((m, n), dtype=torch.int32, device=dev) if Z is None else Z
    if E is None and want_E:
        E = torch.empty((m, n), dtype=torch.float64, device=dev)
    if min_margin is None and want_margin:
        min_margin = torch.empty(1, dtype=torch.float64, device=dev)
    info = torch.zeros(4, dtype=torch.int32, device=dev) if info is None else info
    workspace = _workspace(gptq2d_round_reverse_workspace_bytes(m, n), dev) if workspace is None else workspace
    pX, ldx = _mat(X, torch.float64, "X")
    pL, ldl = _mat(Lr, torch.float64, "Lr")
    pU, ldu = _mat(Ur, torch.float64, "Ur")
    pZ, ldz = _mat(Z, torch.int32, "Z")
    pE, lde = _mat(E, torch.float64, "E")
    st = _lib.gptq2d_round_reverse(m, n, pX, ldx, pL, ldl, pU, ldu, pZ, ldz, pE, lde, _ptr(min_margin),
                                   _ptr(workspace), workspace.numel(), _ptr(info), _stream_ptr(stream))
    if st != OK:
        raise Gptq2dError(st)
    return Z, E, min_margin, info


def gptq2d_round_f32in_workspace_bytes(m, n):
    return int(_lib.gptq2d_round_f32in_workspace_bytes(m, n))


def gptq2d_round_f32in(X, L, U, Z=None, E=None, min_margin=None, workspace=None, info=None, stream=None,
                       want_E=False, want_margin=False):
    """The fp64 sweep on inputs stored in fp32 (float32 CUDA tensors).  Returns (Z, E, min_margin, info)."""
    m, n = X.shape
    dev = X.device
    Z = torch.empty((m, n), dtype=torch.int32, device=dev) if Z is None else Z
    if E is None and want_E:
        E = torch.empty((m, n), dtype=torch.float64, device=dev)
    if min_margin is None and want_margin:
        min_margin = torch.empty(1, dtype=torch.float64, device=dev)
    info = torch.zeros(4, dtype=torch.int32, device=dev) if info is None else info
    workspace = _workspace(gptq2d_round_f32in_workspace_bytes(m, n), dev) if workspace is None else workspace
    pX, ldx = _mat(X, torch.float32, "X")
    pL, ldl = _mat(L, torch.float32, "L")
    pU, ldu = _mat(U, torch.float32, "U")
    pZ, ldz = _mat(Z, torch.int32, "Z")
    pE, lde = _mat(E, torch.float64, "E")
    st = _lib.gptq2d_round_f32in(m, n, pX, ldx, pL, ldl, pU, ldu, pZ, ldz, pE, lde, _ptr(min_margin),
                                 _ptr(workspace), workspace.numel(), _ptr(info), _stream_ptr(stream))
    if st != OK:
        raise Gptq2dError(st)
    return Z, E, min_margin, info


def _factor_problems(As, Bs, Ls, Us, dLs, dUs, shapes):
    count = len(shapes)
    arr = (FactorProblem * count)()
    for b, (m, n) in enumerate(shapes):
        pA, lda = _mat(As[b], torch.float64, "A")
        pB, ldb = _mat(Bs[b], torch.float64, "B")
        pL, ldl = _mat(Ls[b], torch.float64, "L")
        pU, ldu = _mat(Us[b], torch.float64, "U")
        arr[b] = FactorProblem(m, n, pA, lda, pB, ldb, pL, ldl, pU, ldu,
                               _ptr(dLs[b]) if dLs is not None else None, _ptr(dUs[b]) if dUs is not None else None)
    return arr


def make_factor_problems(As, Bs, Ls, Us, dLs=None, dUs=None, shapes=None):
    """The host descriptor array (gptq2d_factor_problem_t[count]) of a batched set-up; reusable across calls
    as long as the tensors it points to stay alive and in place."""
    if shapes is None:
        shapes = [(Ls[b].shape[0], Us[b].shape[0]) for b in range(len(Ls))]
    return _factor_problems(As, Bs, Ls, Us, dLs, dUs, shapes)


def gptq2d_factor_batched_workspace_bytes(problems):
    return int(_lib.gptq2d_factor_batched_workspace_bytes(len(problems), ctypes.cast(problems, ctypes.c_void_p)))


def gptq2d_factor_batched(As=None, Bs=None, shapes=None, Ls=None, Us=None, dLs=None, dUs=None, workspace=None,
                          info=None, stream=None, device=None, problems=None):
    """The set-up of many (A, B) pairs in one call.  As, Bs: sequences of CUDA tensors or None (identity;
    `shapes` = [(m, n), ...] is then needed for those), or `problems` = an array from make_factor_problems
    (the outputs are then whatever that array points to).  Returns (Ls, Us, dLs, dUs, info)."""
    dev = device
    if problems is None:
        count = len(As)
        if shapes is None:
            shapes = [(As[b].shape[0], Bs[b].shape[0]) for b in range(count)]
        if dev is None:
            dev = next((t.device for t in list(As) + list(Bs) if t is not None),
                       torch.device("cuda", torch.cuda.current_device()))
        if Ls is None:
            Ls = [torch.empty((m, m), dtype=torch.float64, device=dev) for (m, n) in shapes]
        if Us is None:
            Us = [torch.empty((n, n), dtype=torch.float64, device=dev) for (m, n) in shapes]
        if dLs is None:
            dLs = [torch.empty(m, dtype=torch.float64, device=dev) for (m, n) in shapes]
        if dUs is None:
            dUs = [torch.empty(n, dtype=torch.float64, device=dev) for (m, n) in shapes]
        problems = _factor_problems(As, Bs, Ls, Us, dLs, dUs, shapes)
    elif dev is None:
        dev = torch.device("cuda", torch.cuda.current_device())
    info = torch.zeros(4, dtype=torch.int32, device=dev) if info is None else info
    if workspace is None:
        workspace = _workspace(gptq2d_factor_batched_workspace_bytes(problems), dev)
    st = _lib.gptq2d_factor_batched(len(problems), ctypes.cast(problems, ctypes.c_void_p), _ptr(workspace),
                                    workspace.numel(), _ptr(info), _stream_ptr(stream))
    if st != OK:
        raise Gptq2dError(st)
    return Ls, Us, dLs, dUs, info


def gptq2d_round_blocked_workspace_bytes(m, n, w):
    return int(_lib.gptq2d_round_blocked_workspace_bytes(m, n, w))


def gptq2d_round_blocked(X, L, U, w, Z=None, E=None, min_margin=None, workspace=None, info=None, stream=None,
                         want_E=False, want_margin=False):
    """Blocked GPTQ-2D (Algorithm 4) with block width w.  Returns (Z, E, min_margin, info)."""
    m, n = X.shape
    dev = X.device
    Z = torch.empty((m, n), dtype=torch.int32, device=dev) if Z is None else Z
    if E is None and want_E:
        E = torch.empty((m, n), dtype=torch.float64, device=dev)
    if min_margin is None and want_margin:
        min_margin = torch.empty(1, dtype=torch.float64, device=dev)
    info = torch.zeros(4, dtype=torch.int32, device=dev) if info is None else info
    if workspace is None:
        workspace = _workspace(gptq2d_round_blocked_workspace_bytes(m, n, w), dev)
    pX, ldx = _mat(X, torch.float64, "X")
    pL, ldl = _mat(L, torch.float64, "L")
    pU, ldu = _mat(U, torch.float64, "U")
    pZ, ldz = _mat(Z, torch.int32, "Z")
    pE, lde = _mat(E, torch.float64, "E")
    st = _lib.gptq2d_round_blocked(m, n, pX, ldx, pL, ldl, pU, ldu, int(w), pZ, ldz, pE, lde, _ptr(min_margin),
                                   _ptr(workspace), workspace.numel(), _ptr(info), _stream_ptr(stream))
    if st != OK:
        raise Gptq2dError(st)
    return Z, E, min_margin, info


def gptq2d_internal_test_hook(key, value):
    """Host-made failure for tests (see the header): 1 = withhold the last copy step of the next pipelined
    host call, 2 = polls after which the wait for a copy step gives up (0: default)."""
    st = _lib.gptq2d_internal_test_hook(int(key), int(value))
    if st != OK:
        raise Gptq2dError(st)


def gptq2d_internal_gemm(A, B, C, transa=False, transb=False, alpha=1.0, beta=0.0, stream=None):
    """C = alpha op(A) op(B) + beta C through the library's own fp64 product (2-D CUDA float64 tensors,
    unit inner stride).  Returns C."""
    M, N = C.shape
    K = A.shape[0] if transa else A.shape[1]
    pA, lda = _mat(A, torch.float64, "A")
    pB, ldb = _mat(B, torch.float64, "B")
    pC, ldc = _mat(C, torch.float64, "C")
    st = _lib.gptq2d_internal_gemm(int(transa), int(transb), M, N, K, float(alpha), pA, lda, pB, ldb, float(beta),
                                   pC, ldc, _stream_ptr(stream))
    if st != OK:
        raise Gptq2dError(st)
    return C


def gptq2d_round_static_max_dim():
    return int(_lib.gptq2d_round_static_max_dim())


def gptq2d_round_static(X, L, U, Z, E=None, min_margin=None, info=None, stream=None):
    """The fp64 sweep for callers that must not allocate: no workspace argument, the library's
    static device array is the scratch (m, n <= gptq2d_round_static_max_dim()).

    Every buffer, Z included, is the caller's: this wrapper creates no tensor either.  All calls
    on a device share the one scratch array, so do not let two of them overlap on the GPU.  The
    first call on a device performs a one-time symbol look-up; issue it before any stream
    capture.  A non-zero C status is raised as Gptq2dError; returns Z."""
    m, n = X.shape
    pX, ldx = _mat(X, torch.float64, "X")
    pL, ldl = _mat(L, torch.float64, "L")
    pU, ldu = _mat(U, torch.float64, "U")
    pZ, ldz = _mat(Z, torch.int32, "Z")
    pE, lde = _mat(E, torch.float64, "E")
    st = _lib.gptq2d_round_static(m, n, pX, ldx, pL, ldl, pU, ldu, pZ, ldz, pE, lde, _ptr(min_margin),
                                  _ptr(info), _stream_ptr(stream))
    if st != OK:
        raise Gptq2dError(st)
    return Z


def _problems(Xs, Ls, Us, Zs, Es):
    count = len(Xs)
    arr = (Problem * count)()
    for b in range(count):
        m, n = Xs[b].shape
        pX, ldx = _mat(Xs[b], torch.float64, "X[%d]" % b)
        pL, ldl = _mat(Ls[b], torch.float64, "L[%d]" % b)
        pU, ldu = _mat(Us[b], torch.float64, "U[%d]" % b)
        pZ, ldz = _mat(Zs[b], torch.int32, "Z[%d]" % b)
        pE, lde = _mat(None if Es is None else Es[b], torch.float64, "E[%d]" % b)
        arr[b] = Problem(m, n, pX.value, ldx, pL.value, ldl, pU.value, ldu, pZ.value, ldz,
                         None if pE is None else pE.value, lde)
    return arr


def make_problems(Xs, Ls, Us, Zs, Es=None):
    """The host descriptor array (gptq2d_problem_t[count]) of a batch; reusable across calls as long as
    the tensors it points to stay alive and in place."""
    return _problems(Xs, Ls, Us, Zs, Es)


def gptq2d_round_batched_workspace_bytes(Xs=None, Ls=None, Us=None, Zs=None, Es=None, problems=None):
    arr = _problems(Xs, Ls, Us, Zs, Es) if problems is None else problems
    return int(_lib.gptq2d_round_batched_workspace_bytes(len(arr), ctypes.cast(arr, ctypes.c_void_p)))


def gptq2d_round_batched(Xs=None, Ls=None, Us=None, Zs=None, Es=None, min_margin=None, workspace=None, info=None,
                         stream=None, want_E=False, want_margin=False, problems=None, device=None):
    """Many independent fp64 sweeps in one launch.  Xs, Ls, Us: sequences of CUDA tensors (shapes may
    differ between matrices), or `problems` = an array from make_problems (then Zs / Es are whatever
    that array points to).  Returns (Zs, Es, min_margin, info); min_margin has one entry per matrix."""
    if problems is None:
        dev = Xs[0].device
        if Zs is None:
            Zs = [torch.empty(tuple(x.shape), dtype=torch.int32, device=dev) for x in Xs]
        if Es is None and want_E:
            Es = [torch.empty(tuple(x.shape), dtype=torch.float64, device=dev) for x in Xs]
        problems = _problems(Xs, Ls, Us, Zs, Es)
    else:
        dev = torch.device("cuda", torch.cuda.current_device()) if device is None else device
    count = len(problems)
    if min_margin is None and want_margin:
        min_margin = torch.empty(count, dtype=torch.float64, device=dev)
    info = torch.zeros(4, dtype=torch.int32, device=dev) if info is None else info
    parr = ctypes.cast(problems, ctypes.c_void_p)
    if workspace is None:
        workspace = _workspace(_lib.gptq2d_round_batched_workspace_bytes(count, parr), dev)
    st = _lib.gptq2d_round_batched(count, parr, _ptr(min_margin), _ptr(workspace), workspace.numel(), _ptr(info),
                                   _stream_ptr(stream))
    if st != OK:
        raise Gptq2dError(st)
    return Zs, Es, min_margin, info


def gptq2d_round_host(hX, hL, hU, hZ=None, hE=None, hmargin=None, precision=FP64, workspace=None, hinfo=None,
                      stream=None, device=None):
    """Host-buffer variant: hX, hL, hU are CPU tensors (pinned for speed); copies in, sweeps, copies Z back,
    synchronises.  Returns (hZ, hinfo)."""
    m, n = hX.shape
    for t, name in ((hX, "hX"), (hL, "hL"), (hU, "hU")):
        if t.is_cuda or t.dtype != torch.float64 or not t.is_contiguous():
            raise ValueError("%s must be a contiguous CPU float64 tensor" % name)
    device = torch.device("cuda", torch.cuda.current_device()) if device is None else device
    hZ = torch.empty((m, n), dtype=torch.int32).pin_memory() if hZ is None else hZ
    hinfo = torch.zeros(4, dtype=torch.int32).pin_memory() if hinfo is None else hinfo
    nbytes = gptq2d_round_host_workspace_bytes(m, n, precision)
    workspace = _workspace(nbytes, device) if workspace is None else workspace
    st = _lib.gptq2d_round_host(m, n, _ptr(hX), _ptr(hL), _ptr(hU), _ptr(hZ), _ptr(hE), _ptr(hmargin),
                                int(precision), _ptr(workspace), workspace.numel(), _ptr(hinfo),
                                _stream_ptr(stream))
    if st != OK:
        raise Gptq2dError(st)
    if int(hinfo[0]) != 0:
        raise Gptq2dError(int(hinfo[0]), hinfo.tolist())
    return hZ, hinfo


def gptq2d_objective(X, Z, A, B, obj=None, workspace=None, info=None, stream=None):
    """|| A (Z - X) B ||_F^2 as a 1-element CUDA tensor.  A or B may be None (identity)."""
    m, n = X.shape
    dev = X.device
    obj = torch.empty(1, dtype=torch.float64, device=dev) if obj is None else obj
    info = torch.zeros(4, dtype=torch.int32, device=dev) if info is None else info
    nbytes = gptq2d_objective_workspace_bytes(m, n)
    workspace = _workspace(nbytes, dev) if workspace is None else workspace
    pX, ldx = _mat(X, torch.float64, "X")
    pZ, ldz = _mat(Z, torch.int32, "Z")
    pA, lda = _mat(A, torch.float64, "A")
    pB, ldb = _mat(B, torch.float64, "B")
    st = _lib.gptq2d_objective(m, n, pX, ldx, pZ, ldz, pA, lda, pB, ldb, _ptr(obj), _ptr(workspace),
                               workspace.numel(), _ptr(info), _stream_ptr(stream))
    if st != OK:
        raise Gptq2dError(st)
    return obj
