"""ctypes front end of the CPU oracle (``matq_ref.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by
the benchmark's CPU-baseline leg, never by the CUDA library or its binding.
All arguments are NumPy host arrays; bf16 tensors are ``uint16`` bit patterns.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "matq_ref.c")
_LIB = os.path.join(_HERE, "libmatq_ref.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_SHAPE = 0, 1, 2, 3
ERR_NONFINITE, ERR_CAPACITY = 8, 9
SRC_BF16, SRC_CODES8, SRC_PACKED = 0, 1, 2


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (strict IEEE: no fast-math, no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fno-fast-math", "-ffp-contract=off", "-fopenmp",
               "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.matq_ref_num_threads.restype = C.c_int
    return _lib


def num_threads() -> int:
    return int(lib().matq_ref_num_threads())


def _p(a, ctype=C.c_void_p):
    return None if a is None else a.ctypes.data_as(ctype)


def _chk(a, dtype, name):
    assert isinstance(a, np.ndarray) and a.dtype == dtype and a.flags.c_contiguous, name
    return a


def quantize(W_bits: np.ndarray, c: int = 8, want_codes: bool = True):
    """Eq. 1 per row.  Returns (status, q uint8 [N,K] or None, alpha f32 [N], zero f32 [N])."""
    _chk(W_bits, np.uint16, "W")
    N, K = W_bits.shape
    q = np.empty((N, K), np.uint8) if want_codes else None
    alpha = np.zeros(N, np.float32)
    zero = np.zeros(N, np.float32)
    st = lib().matq_ref_quantize(_p(W_bits), C.c_int64(N), C.c_int64(K), C.c_int64(K), C.c_int(c),
                                 _p(q), _p(alpha), _p(zero))
    return st, q, alpha, zero


def quantize_clip(W_bits: np.ndarray, gamma=None, beta=None, c: int = 8, want_codes: bool = True):
    """Eq. 3 per row (gamma, beta fp32 [N] or None = 1).  Returns (status, q or None, alpha, zero)."""
    _chk(W_bits, np.uint16, "W")
    N, K = W_bits.shape
    if gamma is not None:
        _chk(gamma, np.float32, "gamma")
    if beta is not None:
        _chk(beta, np.float32, "beta")
    q = np.empty((N, K), np.uint8) if want_codes else None
    alpha = np.zeros(N, np.float32)
    zero = np.zeros(N, np.float32)
    st = lib().matq_ref_quantize_clip(_p(W_bits), C.c_int64(N), C.c_int64(K), C.c_int64(K), C.c_int(c),
                                      _p(gamma), _p(beta), _p(q), _p(alpha), _p(zero))
    return st, q, alpha, zero


def slice_values(q: np.ndarray, r: int, extra_precision: bool = False, c: int = 8):
    """Eq. 6 (or Eq. 8) elementwise.  Returns (status, S uint16, same shape)."""
    _chk(q, np.uint8, "q")
    S = np.empty(q.shape, np.uint16)
    st = lib().matq_ref_slice(_p(q), C.c_int64(q.size), C.c_int(c), C.c_int(r),
                              C.c_int(int(extra_precision)), _p(S))
    return st, S


def slice_pack(q: np.ndarray, r: int, extra_precision: bool = False, c: int = 8,
               ovf_capacity: int | None = None, want_packed: bool = True, want_unpacked: bool = True):
    """Returns dict(status, packed, sliced, ovf_row_ptr, ovf_col, ovf_count)."""
    _chk(q, np.uint8, "q")
    N, K = q.shape
    packable = r in (8, 4, 2)
    packed = np.zeros((N, K * r // 8), np.uint8) if (want_packed and packable) else None
    sliced = np.zeros((N, K), np.uint8) if want_unpacked else None
    ep = bool(extra_precision) and r < c
    cap = N * K if ovf_capacity is None else int(ovf_capacity)
    row_ptr = np.zeros(N + 1, np.int32) if ep else None
    col = np.zeros(max(cap, 1), np.uint16) if ep else None
    cnt = C.c_int64(0)
    st = lib().matq_ref_slice_pack(_p(q), C.c_int64(N), C.c_int64(K), C.c_int(c), C.c_int(r),
                                   C.c_int(int(extra_precision)), _p(packed), _p(sliced),
                                   _p(row_ptr), _p(col), C.c_int64(cap), C.byref(cnt))
    if ep and st == OK:
        col = col[:cnt.value].copy()
    return dict(status=st, packed=packed, sliced=sliced, ovf_row_ptr=row_ptr, ovf_col=col,
                ovf_count=int(cnt.value))


def unpack(packed: np.ndarray, K: int, r: int):
    _chk(packed, np.uint8, "packed")
    N = packed.shape[0]
    fields = np.empty((N, K), np.uint8)
    st = lib().matq_ref_unpack(_p(packed), C.c_int64(N), C.c_int64(K), C.c_int(r), _p(fields))
    return st, fields


def gemv(packed: np.ndarray, K: int, r: int, alpha: np.ndarray, zero: np.ndarray,
         x_bits: np.ndarray, ovf_row_ptr=None, ovf_col=None, c: int = 8):
    """y = x . dequant(S)^T in fp64.  Returns (status, y float64 [B, N])."""
    _chk(packed, np.uint8, "packed"); _chk(alpha, np.float32, "alpha"); _chk(zero, np.float32, "zero")
    _chk(x_bits, np.uint16, "x")
    N = packed.shape[0]
    B = x_bits.shape[0]
    assert x_bits.shape[1] == K
    y = np.zeros((B, N), np.float64)
    S = np.empty((N, K), np.uint16)
    if ovf_col is not None and ovf_col.size == 0:
        ovf_col = np.zeros(1, np.uint16)
    st = lib().matq_ref_gemv(_p(packed), C.c_int64(N), C.c_int64(K), C.c_int(c), C.c_int(r),
                             _p(alpha), _p(zero), _p(ovf_row_ptr), _p(ovf_col),
                             _p(x_bits), C.c_int64(B), C.c_int64(K), _p(y), C.c_int64(N), _p(S))
    return st, y


def gemm_multi(src_kind: int, Wsrc: np.ndarray, K: int, X_bits: np.ndarray, rs=(8, 4, 2),
               alpha=None, zero=None, extra_precision: bool = False,
               ovf_row_ptr=None, ovf_col=None, c: int = 8):
    """Forward at every precision in ``rs`` (Eq. 7's F(S(Q(W, c), r), x)).
    Returns (status, [Y_r float64 [M, N]], alpha, zero)."""
    N = Wsrc.shape[0]
    M = X_bits.shape[0]
    _chk(X_bits, np.uint16, "X")
    assert X_bits.shape[1] == K
    if src_kind == SRC_BF16:
        _chk(Wsrc, np.uint16, "W")
        alpha = np.zeros(N, np.float32)
        zero = np.zeros(N, np.float32)
    else:
        _chk(Wsrc, np.uint8, "Wsrc")
        _chk(alpha, np.float32, "alpha"); _chk(zero, np.float32, "zero")
    Ys = [np.zeros((M, N), np.float64) for _ in rs]
    Yp = (C.c_void_p * len(rs))(*[y.ctypes.data for y in Ys])
    rs_arr = (C.c_int * len(rs))(*rs)
    qs = np.empty((N, K), np.uint8)
    S = np.empty((N, K), np.uint16)
    if ovf_col is not None and ovf_col.size == 0:
        ovf_col = np.zeros(1, np.uint16)
    st = lib().matq_ref_gemm_multi(C.c_int(src_kind), _p(Wsrc), C.c_int64(N), C.c_int64(K), C.c_int(c),
                                   _p(alpha), _p(zero), C.c_int(int(extra_precision)),
                                   _p(ovf_row_ptr), _p(ovf_col), _p(X_bits), C.c_int64(M), C.c_int64(K),
                                   rs_arr, C.c_int(len(rs)), Yp, C.c_int64(N), _p(qs), _p(S))
    return st, Ys, alpha, zero


TEACHER_AND_TARGET = 256


def gemm_multi_loss(src_kind: int, Wsrc: np.ndarray, K: int, X_bits: np.ndarray, Yt: np.ndarray, lambdas, rs=(8, 4, 2),
                    alpha=None, zero=None, extra_precision: bool = False, ovf_row_ptr=None, ovf_col=None, c: int = 8,
                    teacher=None):
    """Eq. 7 with the L2 reconstruction loss of Eq. 5 for one linear layer: for every r in ``rs``
    L_r = sum over tokens and channels of (Yt - F(S(Q(W, c), r), X))^2 against a given target Yt (fp32 [M, N], e.g. the
    bf16 layer's output), and the weighted objective sum_r lambda_r L_r (no 1/N: the caller divides by its sample count).
    The definition written out with NumPy in float64 on top of ``gemm_multi``.
    Returns (status, [L_r], total, alpha, zero)."""
    assert Yt.dtype == np.float32 and len(lambdas) == len(rs)
    st, Ys, alpha, zero = gemm_multi(src_kind, Wsrc, K, X_bits, rs=rs, alpha=alpha, zero=zero,
                                     extra_precision=extra_precision, ovf_row_ptr=ovf_row_ptr, ovf_col=ovf_col, c=c)
    if st != OK:
        return st, None, None, alpha, zero
    t = Yt.astype(np.float64)
    losses = []
    for i, y in enumerate(Ys):
        # co-distillation (Section 5.2): teacher[i] = j >= 0 replaces the target of precision i by the output of the
        # higher-precision nested model rs[j]; j + TEACHER_AND_TARGET uses both, weighted equally; -1 = target only
        code = -1 if teacher is None else int(teacher[i])
        L = 0.0
        if code < 0 or code >= TEACHER_AND_TARGET:
            L += float(((t - y) ** 2).sum())
        if code >= 0:
            L += float(((Ys[code % TEACHER_AND_TARGET] - y) ** 2).sum())
        losses.append(L)
    total = float(sum(float(l) * L for l, L in zip(lambdas, losses)))
    return st, losses, total, alpha, zero
