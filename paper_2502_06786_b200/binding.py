"""Thin ctypes binding over the C ABI declared in ``include/matq.h``.

Argument marshalling only: every function checks device / dtype / layout of
its torch tensors, passes raw device pointers and the current CUDA stream to
the library and returns the outputs.  No arithmetic of the method happens in
Python, and there is no CPU fallback: if the shared library is missing the
import of this module fails.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libmatq.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_SHAPE, ERR_ALIGNMENT = 0, 1, 2, 3, 4
ERR_WORKSPACE, ERR_CUDA, ERR_NONFINITE, ERR_CAPACITY, ERR_TIMEOUT = 5, 6, 8, 9, 10
SRC_BF16, SRC_CODES8, SRC_PACKED = 0, 1, 2
GEMV_AUTO, GEMV_CUDA_CORE, GEMV_TENSOR, GEMV_TCGEN05, GEMV_TENSOR_INT8, GEMV_STREAM, GEMV_PDL = 0, 1, 2, 3, 4, 5, 0x100
GEMV_TEST_STALL = 0x8000
TEACHER_AND_TARGET = 256    # matq_gemm_multi_loss: teacher[i] = TEACHER_AND_TARGET + j

EXPORTS = ["matq_status_string", "matq_version", "matq_packed_row_bytes", "matq_quantize", "matq_quantize_clip",
           "matq_slice_pack", "matq_slice_pack_nested", "matq_gemv_workspace_bytes", "matq_gemv", "matq_gemv_grouped", "matq_gemv_grouped_launches",
           "matq_gemm_multi_workspace_bytes", "matq_gemm_multi",
           "matq_gemm_multi_loss_workspace_bytes", "matq_gemm_multi_loss",
           "matq_gemm_multi_test_stall", "matq_slice_pack_test_stall",
           "matq_gemm_multi_static_max_bytes", "matq_gemm_multi_static"]


class GemvProblem(C.Structure):
    """matq_gemv_problem."""
    _fields_ = [("packed", C.c_void_p), ("N", C.c_int64), ("K", C.c_int64), ("r", C.c_int),
                ("alpha", C.c_void_p), ("zero", C.c_void_p), ("ovf_row_ptr", C.c_void_p), ("ovf_col", C.c_void_p),
                ("x", C.c_void_p), ("y", C.c_void_p), ("B", C.c_int64)]


class MatqError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (status {status})")


def _load():
    if not os.path.exists(_LIB_PATH):
        raise ImportError(
            f"{_LIB_PATH} is missing: build it with `python -m paper_2502_06786_b200.build` "
            "(there is no fallback implementation)")
    lib = C.CDLL(_LIB_PATH)
    i64, i32, vp, sz, u32 = C.c_int64, C.c_int, C.c_void_p, C.c_size_t, C.c_uint
    lib.matq_status_string.restype = C.c_char_p
    lib.matq_status_string.argtypes = [i32]
    lib.matq_version.restype = i32
    lib.matq_packed_row_bytes.restype = i64
    lib.matq_packed_row_bytes.argtypes = [i64, i32]
    lib.matq_quantize.restype = i32
    lib.matq_quantize.argtypes = [vp, i64, i64, i64, i32, vp, vp, vp, vp, vp]
    lib.matq_quantize_clip.restype = i32
    lib.matq_quantize_clip.argtypes = [vp, i64, i64, i64, i32, vp, vp, vp, vp, vp, vp, vp]
    lib.matq_slice_pack.restype = i32
    lib.matq_slice_pack.argtypes = [vp, i64, i64, i32, i32, i32, vp, vp, vp, vp, i64, vp, vp, vp]
    lib.matq_slice_pack_nested.restype = i32
    lib.matq_slice_pack_nested.argtypes = [vp, i64, i64, i32, vp, vp, i32, vp, vp, i64, vp, vp, vp]
    lib.matq_gemv_workspace_bytes.restype = sz
    lib.matq_gemv_workspace_bytes.argtypes = [i64, i64, i32, i32]
    lib.matq_gemv.restype = i32
    lib.matq_gemv.argtypes = [vp, i64, i64, i32, i32, vp, vp, vp, vp, vp, i32, i64, vp, i64, vp, sz, u32, vp, vp]
    lib.matq_gemv_grouped.restype = i32
    lib.matq_gemv_grouped.argtypes = [C.POINTER(GemvProblem), i32, i32, u32, vp, vp]
    lib.matq_gemv_grouped_launches.restype = i32
    lib.matq_gemv_grouped_launches.argtypes = [C.POINTER(GemvProblem), i32]
    lib.matq_gemm_multi_workspace_bytes.restype = sz
    lib.matq_gemm_multi_workspace_bytes.argtypes = [i32, i64, i64, i64, i32]
    lib.matq_gemm_multi.restype = i32
    lib.matq_gemm_multi.argtypes = [i32, vp, i64, i64, i32, vp, vp, i32, vp, vp, vp, i64, i64,
                                    C.POINTER(C.c_int), i32, C.POINTER(C.c_void_p), i64, vp, sz, vp, vp]
    lib.matq_gemm_multi_loss_workspace_bytes.restype = sz
    lib.matq_gemm_multi_loss_workspace_bytes.argtypes = [i32, i64, i64, i64, i32]
    lib.matq_gemm_multi_loss.restype = i32
    lib.matq_gemm_multi_loss.argtypes = [i32, vp, i64, i64, i32, vp, vp, i32, vp, vp, vp, i64, i64,
                                         C.POINTER(C.c_int), i32, C.POINTER(C.c_float), C.POINTER(C.c_int), vp, i64, vp, vp, sz, vp, vp]
    lib.matq_gemm_multi_test_stall.restype = i32
    lib.matq_gemm_multi_test_stall.argtypes = [i32]
    lib.matq_slice_pack_test_stall.restype = i32
    lib.matq_slice_pack_test_stall.argtypes = [i32]
    lib.matq_gemm_multi_static_max_bytes.restype = sz
    lib.matq_gemm_multi_static_max_bytes.argtypes = []
    lib.matq_gemm_multi_static.restype = i32
    lib.matq_gemm_multi_static.argtypes = [i32, vp, i64, i64, i32, vp, vp, i32, vp, vp, vp, i64, i64,
                                           C.POINTER(C.c_int), i32, C.POINTER(C.c_void_p), i64, vp, vp]
    return lib


_lib = _load()


def lib_path() -> str:
    return _LIB_PATH


def status_string(status: int) -> str:
    return _lib.matq_status_string(int(status)).decode()


def version() -> int:
    return int(_lib.matq_version())


def packed_row_bytes(K: int, r: int) -> int:
    return int(_lib.matq_packed_row_bytes(K, r))


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _dev(t, dtype, name, ndim=None):
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.dtype == dtype):
        raise TypeError(f"{name}: expected a CUDA tensor of dtype {dtype}")
    if ndim is not None and t.dim() != ndim:
        raise ValueError(f"{name}: expected {ndim} dimensions")
    return t


def _ld(t, inner):
    """Row stride in elements of a 2-D tensor (a single row may report any stride)."""
    return t.stride(0) if t.shape[0] > 1 else max(inner, t.stride(0))


def _check(st, where, raise_on_error=True):
    if st != OK and raise_on_error:
        raise MatqError(st, where)
    return st


def quantize(W, q=None, alpha=None, zero=None, dev_status=None, want_codes=True, c=8, gamma=None, beta=None):
    """matq_quantize, or matq_quantize_clip when gamma / beta (fp32 [N], Eq. 3's clipping scales) are given.
    W: bf16 [N, K] (row stride W.stride(0)).  Returns (q, alpha, zero)."""
    _dev(W, torch.bfloat16, "W", 2)
    if W.stride(1) != 1:
        raise ValueError("W: unit stride along K required")
    N, K = W.shape
    dev = W.device
    if q is None and want_codes:
        q = torch.empty((N, K), dtype=torch.uint8, device=dev)
    if alpha is None:
        alpha = torch.empty(N, dtype=torch.float32, device=dev)
    if zero is None:
        zero = torch.empty(N, dtype=torch.float32, device=dev)
    if gamma is None and beta is None:
        st = _lib.matq_quantize(_ptr(W), N, K, _ld(W, K), c, _ptr(q), _ptr(alpha), _ptr(zero),
                                _ptr(dev_status), _stream())
        _check(st, "matq_quantize")
    else:
        for name, t in (("gamma", gamma), ("beta", beta)):
            if t is not None:
                _dev(t, torch.float32, name, 1)
                if t.numel() != N or not t.is_contiguous():
                    raise ValueError(f"{name}: contiguous fp32 [N] required")
        st = _lib.matq_quantize_clip(_ptr(W), N, K, _ld(W, K), c, _ptr(gamma), _ptr(beta), _ptr(q), _ptr(alpha),
                                     _ptr(zero), _ptr(dev_status), _stream())
        _check(st, "matq_quantize_clip")
    return q, alpha, zero


def slice_pack(q, r, extra_precision=False, packed=None, sliced_unpacked=None, ovf_row_ptr=None, ovf_col=None,
               ovf_capacity=None, ovf_count=None, dev_status=None, want_packed=True, want_unpacked=False, c=8,
               raise_on_error=True):
    """matq_slice_pack.  Returns dict(status, packed, sliced, ovf_row_ptr, ovf_col, ovf_count)."""
    _dev(q, torch.uint8, "q", 2)
    if not q.is_contiguous():
        raise ValueError("q must be contiguous")
    N, K = q.shape
    dev = q.device
    if packed is None and want_packed:
        packed = torch.empty((N, max(K * r // 8, 0)), dtype=torch.uint8, device=dev)
    if sliced_unpacked is None and want_unpacked:
        sliced_unpacked = torch.empty((N, K), dtype=torch.uint8, device=dev)
    ep = bool(extra_precision) and r < c
    if ep:
        if ovf_row_ptr is None:
            ovf_row_ptr = torch.empty(N + 1, dtype=torch.int32, device=dev)
        if ovf_capacity is None:
            ovf_capacity = ovf_col.numel() if ovf_col is not None else N * K
        if ovf_col is None:
            ovf_col = torch.empty(max(ovf_capacity, 1), dtype=torch.uint16, device=dev)
        if ovf_count is None:
            ovf_count = torch.zeros(1, dtype=torch.int64, device=dev)
    st = _lib.matq_slice_pack(_ptr(q), N, K, c, r, int(bool(extra_precision)), _ptr(packed), _ptr(sliced_unpacked),
                              _ptr(ovf_row_ptr), _ptr(ovf_col), int(ovf_capacity or 0), _ptr(ovf_count),
                              _ptr(dev_status), _stream())
    _check(st, "matq_slice_pack", raise_on_error)
    return dict(status=st, packed=packed, sliced=sliced_unpacked, ovf_row_ptr=ovf_row_ptr, ovf_col=ovf_col,
                ovf_count=ovf_count)


def slice_pack_nested(q, extra_precision=True, packed4=None, packed2=None, ovf_row_ptr=None, ovf_col=None, ovf_capacity=None,
                      ovf_count=None, dev_status=None, c=8, raise_on_error=True):
    """matq_slice_pack_nested.  Returns dict(status, packed4, packed2, ovf_row_ptr, ovf_col, ovf_count)."""
    _dev(q, torch.uint8, "q", 2)
    if not q.is_contiguous():
        raise ValueError("q must be contiguous")
    N, K = q.shape
    dev = q.device
    if packed4 is None:
        packed4 = torch.empty((N, K // 2), dtype=torch.uint8, device=dev)
    if packed2 is None:
        packed2 = torch.empty((N, K // 4), dtype=torch.uint8, device=dev)
    if extra_precision:
        if ovf_row_ptr is None:
            ovf_row_ptr = torch.empty(N + 1, dtype=torch.int32, device=dev)
        if ovf_capacity is None:
            ovf_capacity = ovf_col.numel() if ovf_col is not None else N * K
        if ovf_col is None:
            ovf_col = torch.empty(max(ovf_capacity, 1), dtype=torch.uint16, device=dev)
        if ovf_count is None:
            ovf_count = torch.zeros(1, dtype=torch.int64, device=dev)
    st = _lib.matq_slice_pack_nested(_ptr(q), N, K, c, _ptr(packed4), _ptr(packed2), int(bool(extra_precision)),
                                     _ptr(ovf_row_ptr), _ptr(ovf_col), int(ovf_capacity or 0), _ptr(ovf_count),
                                     _ptr(dev_status), _stream())
    _check(st, "matq_slice_pack_nested", raise_on_error)
    return dict(status=st, packed4=packed4, packed2=packed2, ovf_row_ptr=ovf_row_ptr, ovf_col=ovf_col, ovf_count=ovf_count)


def gemv_workspace_bytes(N, K, r, B) -> int:
    return int(_lib.matq_gemv_workspace_bytes(N, K, r, B))


def gemv(packed, K, r, alpha, zero, x, y=None, ovf_row_ptr=None, ovf_col=None, workspace=None, flags=GEMV_AUTO,
         dev_status=None, c=8):
    """matq_gemv.  packed: uint8 [N, K*r/8]; x: bf16 [B, K]; returns y fp32 [B, N]."""
    _dev(packed, torch.uint8, "packed", 2)
    _dev(x, torch.bfloat16, "x", 2)
    _dev(alpha, torch.float32, "alpha"); _dev(zero, torch.float32, "zero")
    if not packed.is_contiguous() or x.stride(1) != 1:
        raise ValueError("packed must be contiguous and x unit-stride along K")
    N = packed.shape[0]
    B = x.shape[0]
    if y is None:
        y = torch.empty((B, N), dtype=torch.float32, device=packed.device)
    need = gemv_workspace_bytes(N, K, r, B)
    if workspace is None and need:
        workspace = torch.empty(need, dtype=torch.uint8, device=packed.device)
    st = _lib.matq_gemv(_ptr(packed), N, K, c, r, _ptr(alpha), _ptr(zero), _ptr(ovf_row_ptr), _ptr(ovf_col),
                        _ptr(x), B, _ld(x, K), _ptr(y), _ld(y, N),
                        _ptr(workspace), workspace.numel() if workspace is not None else 0, int(flags),
                        _ptr(dev_status), _stream())
    _check(st, "matq_gemv")
    return y


def gemv_group(problems):
    """Descriptor array for gemv_grouped from dicts / tuples (packed, K, r, alpha, zero, x, y[, ovf_row_ptr, ovf_col]).
    x [K] with y [N] is one activation vector; x [B, K] with y [B, N] (2 <= B <= 16, dense rows) a batch.
    Build it once and reuse it: it holds raw pointers, the caller keeps the tensors alive."""
    arr = (GemvProblem * len(problems))()
    for d, pr in zip(arr, problems):
        if isinstance(pr, dict):
            pr = (pr["packed"], pr["K"], pr["r"], pr["alpha"], pr["zero"], pr["x"], pr["y"], pr.get("ovf_row_ptr"), pr.get("ovf_col"))
        packed, K, r, alpha, zero, x, y = pr[:7]
        rp, col = (pr[7], pr[8]) if len(pr) > 7 else (None, None)
        _dev(packed, torch.uint8, "packed", 2); _dev(x, torch.bfloat16, "x"); _dev(y, torch.float32, "y")
        _dev(alpha, torch.float32, "alpha"); _dev(zero, torch.float32, "zero")
        N = packed.shape[0]
        B = x.shape[0] if x.dim() == 2 and x.shape[0] > 1 else 1
        if not packed.is_contiguous() or not x.is_contiguous() or not y.is_contiguous() or x.numel() != B * K or y.numel() != B * N:
            raise ValueError("packed, x [K] or [B, K] and y [N] or [B, N] must be contiguous and match the shape")
        d.packed, d.N, d.K, d.r = packed.data_ptr(), N, K, r
        d.alpha, d.zero, d.x, d.y = alpha.data_ptr(), zero.data_ptr(), x.data_ptr(), y.data_ptr()
        d.ovf_row_ptr = None if rp is None else rp.data_ptr()
        d.ovf_col = None if col is None else col.data_ptr()
        d.B = B
    return arr


def gemv_grouped(group, flags=0, dev_status=None, c=8, raise_on_error=True):
    """matq_gemv_grouped on a descriptor array from gemv_group (or a list accepted by it)."""
    if not isinstance(group, C.Array):
        group = gemv_group(group)
    st = _lib.matq_gemv_grouped(group, len(group), c, int(flags), _ptr(dev_status), _stream())
    _check(st, "matq_gemv_grouped", raise_on_error)
    return st


def gemv_grouped_launches(group) -> int:
    """Kernel launches gemv_grouped makes for this descriptor array."""
    if not isinstance(group, C.Array):
        group = gemv_group(group)
    return int(_lib.matq_gemv_grouped_launches(group, len(group)))


def gemm_multi_workspace_bytes(src_kind, M, N, K, n_r) -> int:
    return int(_lib.matq_gemm_multi_workspace_bytes(src_kind, M, N, K, n_r))


def gemm_multi(src_kind, Wsrc, K, X, rs=(8, 4, 2), alpha=None, zero=None, extra_precision=False,
               ovf_row_ptr=None, ovf_col=None, Ys=None, workspace=None, dev_status=None, c=8):
    """matq_gemm_multi.  Returns (Ys, alpha, zero); Ys[i] is fp32 [M, N] for rs[i]."""
    _dev(X, torch.bfloat16, "X", 2)
    _dev(Wsrc, torch.bfloat16 if src_kind == SRC_BF16 else torch.uint8, "Wsrc", 2)
    N = Wsrc.shape[0]
    M = X.shape[0]
    dev = X.device
    if alpha is None:
        alpha = torch.empty(N, dtype=torch.float32, device=dev)
    if zero is None:
        zero = torch.empty(N, dtype=torch.float32, device=dev)
    if Ys is None:
        Ys = [torch.empty((M, N), dtype=torch.float32, device=dev) for _ in rs]
    need = gemm_multi_workspace_bytes(src_kind, M, N, K, len(rs))
    if workspace is None and need:
        workspace = torch.empty(need, dtype=torch.uint8, device=dev)
    rs_arr = (C.c_int * len(rs))(*rs)
    y_arr = (C.c_void_p * len(rs))(*[y.data_ptr() for y in Ys])
    st = _lib.matq_gemm_multi(src_kind, _ptr(Wsrc), N, K, c, _ptr(alpha), _ptr(zero), int(bool(extra_precision)),
                              _ptr(ovf_row_ptr), _ptr(ovf_col), _ptr(X), M, _ld(X, K), rs_arr, len(rs),
                              y_arr, _ld(Ys[0], N), _ptr(workspace),
                              workspace.numel() if workspace is not None else 0, _ptr(dev_status), _stream())
    _check(st, "matq_gemm_multi")
    return Ys, alpha, zero


def gemm_multi_loss_workspace_bytes(src_kind, M, N, K, n_r) -> int:
    return int(_lib.matq_gemm_multi_loss_workspace_bytes(src_kind, M, N, K, n_r))


def gemm_multi_loss(src_kind, Wsrc, K, X, Yt, lambdas, rs=(8, 4, 2), alpha=None, zero=None, extra_precision=False,
                    ovf_row_ptr=None, ovf_col=None, loss=None, workspace=None, dev_status=None, c=8, teacher=None):
    """matq_gemm_multi_loss.  Yt: fp32 [M, N] target.  Returns (loss, alpha, zero); loss is a device float64 tensor
    [len(rs) + 1]: one squared error per precision and the lambda-weighted total."""
    _dev(X, torch.bfloat16, "X", 2)
    _dev(Yt, torch.float32, "Yt", 2)
    _dev(Wsrc, torch.bfloat16 if src_kind == SRC_BF16 else torch.uint8, "Wsrc", 2)
    if len(lambdas) != len(rs):
        raise ValueError("one lambda per precision")
    N = Wsrc.shape[0]
    M = X.shape[0]
    dev = X.device
    if Yt.shape != (M, N) or Yt.stride(1) != 1:
        raise ValueError("Yt: fp32 [M, N] with unit stride along N required")
    if alpha is None:
        alpha = torch.empty(N, dtype=torch.float32, device=dev)
    if zero is None:
        zero = torch.empty(N, dtype=torch.float32, device=dev)
    if loss is None:
        loss = torch.empty(len(rs) + 1, dtype=torch.float64, device=dev)
    need = gemm_multi_loss_workspace_bytes(src_kind, M, N, K, len(rs))
    if workspace is None and need:
        workspace = torch.empty(need, dtype=torch.uint8, device=dev)
    rs_arr = (C.c_int * len(rs))(*rs)
    lam = (C.c_float * len(rs))(*[float(v) for v in lambdas])
    tch = (C.c_int * len(rs))(*[int(v) for v in teacher]) if teacher is not None else None
    st = _lib.matq_gemm_multi_loss(src_kind, _ptr(Wsrc), N, K, c, _ptr(alpha), _ptr(zero), int(bool(extra_precision)),
                                   _ptr(ovf_row_ptr), _ptr(ovf_col), _ptr(X), M, _ld(X, K), rs_arr, len(rs), lam, tch,
                                   _ptr(Yt), _ld(Yt, N), _ptr(loss), _ptr(workspace),
                                   workspace.numel() if workspace is not None else 0, _ptr(dev_status), _stream())
    _check(st, "matq_gemm_multi_loss")
    return loss, alpha, zero


def slice_pack_test_stall(on) -> int:
    """matq_slice_pack_test_stall: switch the one-pass slice kernel's "first tile never publishes" test mode."""
    return int(_lib.matq_slice_pack_test_stall(1 if on else 0))


def gemm_multi_test_stall(on) -> int:
    """matq_gemm_multi_test_stall: switch the dense kernel's "issue no copies" test mode; returns the previous setting."""
    return int(_lib.matq_gemm_multi_test_stall(1 if on else 0))


def gemm_multi_static_max_bytes() -> int:
    return int(_lib.matq_gemm_multi_static_max_bytes())


def gemm_multi_static(src_kind, Wsrc, K, X, Ys, alpha, zero, rs=(8, 4, 2), extra_precision=False,
                      ovf_row_ptr=None, ovf_col=None, dev_status=None, c=8, raise_on_error=True):
    """matq_gemm_multi_static: the dense forward with the library's built-in scratch.

    For callers that cannot allocate device memory at call time.  Unlike ``gemm_multi`` this wrapper allocates
    nothing either: the outputs ``Ys`` (one fp32 [M, N] tensor per precision), ``alpha`` and ``zero`` must be passed in.
    Returns the status (raises ``MatqError`` unless ``raise_on_error`` is false).
    """
    _dev(X, torch.bfloat16, "X", 2)
    _dev(Wsrc, torch.bfloat16 if src_kind == SRC_BF16 else torch.uint8, "Wsrc", 2)
    N, M = Wsrc.shape[0], X.shape[0]
    rs_arr = (C.c_int * len(rs))(*rs)
    y_arr = (C.c_void_p * len(rs))(*[y.data_ptr() for y in Ys])
    st = _lib.matq_gemm_multi_static(src_kind, _ptr(Wsrc), N, K, c, _ptr(alpha), _ptr(zero), int(bool(extra_precision)),
                                     _ptr(ovf_row_ptr), _ptr(ovf_col), _ptr(X), M, _ld(X, K), rs_arr, len(rs),
                                     y_arr, _ld(Ys[0], N), _ptr(dev_status), _stream())
    return _check(st, "matq_gemm_multi_static", raise_on_error)
