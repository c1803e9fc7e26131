"""CPU oracle (fp64, plain definition) for the fused GEMM + epilogue + row-reduce operator.

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the
benchmark's CPU-baseline leg.  The CUDA package never imports it and shares no
code with it.  The arithmetic lives in ``fgr_oracle.c`` (three nested loops);
this file only compiles it with gcc and marshals numpy arrays through ctypes.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "fgr_oracle.c")
_LIB = os.path.join(_HERE, "libfgr_oracle.so")

F32, BF16 = 0, 1
ACT_NONE, ACT_RELU, ACT_GELU_TANH, ACT_SIGMOID, ACT_TANH, ACT_SILU = 0, 1, 2, 3, 4, 5
SCALE_NONE, SCALE_SCALAR, SCALE_PER_COLUMN = 0, 1, 2
RED_LSE, RED_SOFTMAX, RED_MAXSUM, RED_MAX_SUMEXP = 0, 1, 2, 3
RED_MAX, RED_SUM = 4, 5          # stand-alone reduction only
RED_MEANVAR = 6                  # (mean, population variance) of y over N


class _Problem(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int32), ("M", ctypes.c_int32), ("N", ctypes.c_int32), ("K", ctypes.c_int32),
                ("dtype", ctypes.c_int32), ("act", ctypes.c_int32), ("scale_kind", ctypes.c_int32),
                ("reduce", ctypes.c_int32), ("scale", ctypes.c_double), ("bias_per_batch", ctypes.c_int32),
                ("reserved", ctypes.c_int32)]


def build(force: bool = False) -> str:
    """Compiles ``fgr_oracle.c`` into ``libfgr_oracle.so`` next to it (gcc, strict fp64: no contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.run(["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fopenmp", "-fPIC", "-shared",
                        "-o", tmp, _SRC, "-lm"], check=True)
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.fgr_oracle_rows.restype = ctypes.c_int
        _lib.fgr_oracle_rows.argtypes = [ctypes.POINTER(_Problem)] + [ctypes.c_void_p] * 5 + [
            ctypes.c_int64, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int]
        _lib.fgr_oracle_rows_residual.restype = ctypes.c_int
        _lib.fgr_oracle_rows_residual.argtypes = [ctypes.POINTER(_Problem)] + [ctypes.c_void_p] * 6 + [
            ctypes.c_int64, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int]
        _lib.fgr_oracle_reduce_rows.restype = ctypes.c_int
        _lib.fgr_oracle_reduce_rows.argtypes = [ctypes.c_int32] * 4 + [ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p,
                                                ctypes.c_void_p]
        _lib.fgr_oracle_gelu_tanh.restype = ctypes.c_double
        _lib.fgr_oracle_gelu_tanh.argtypes = [ctypes.c_double]
        _lib.fgr_oracle_act.restype = ctypes.c_double
        _lib.fgr_oracle_act.argtypes = [ctypes.c_int, ctypes.c_double]
    return _lib


def gelu_tanh(u: float) -> float:
    return lib().fgr_oracle_gelu_tanh(float(u))


def act(kind: int, u: float) -> float:
    return lib().fgr_oracle_act(int(kind), float(u))


def out_width(reduce: int) -> int:
    return {RED_LSE: 1, RED_SOFTMAX: 0, RED_MAXSUM: 2, RED_MAX_SUMEXP: 2, RED_MEANVAR: 2}[reduce]


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def run(X, W, bias, scale_vec, *, dtype, act, scale_kind, reduce, scale=1.0, bias_per_batch=0,
        rows=None, want_y=True, nthreads=0, residual=None):
    """Evaluates the operator's definition in fp64.

    X [batch, M, K] and W [batch, N, K] (2-D arrays are taken as batch 1; a W of batch 1 is used for
    every batch element of X): fp32 values
    (``dtype == F32``) or uint16 bf16 bit patterns (``dtype == BF16``).  ``bias`` fp32 [N]
    (or [batch, N] with ``bias_per_batch``) or None; ``scale_vec`` fp32 [N] or None.
    ``rows``: global row indices (bt * M + m) to evaluate; None = all rows.
    ``residual``: R [batch, M, N] in the dtype of X (fp32 values or bf16 bit patterns), added to y
    after the scale, or None.

    Returns ``(Y, out, threads)``: Y fp64 [nrows, N] (y, or P for SOFTMAX; None unless
    ``want_y``), out fp64 [nrows, width] (None for SOFTMAX), threads used.
    """
    want = np.float32 if dtype == F32 else np.uint16
    X = np.ascontiguousarray(X)
    W = np.ascontiguousarray(W)
    if X.dtype != want or W.dtype != want:
        raise TypeError("X/W must be %s for dtype %d" % (want.__name__, dtype))
    if X.ndim == 2:
        X = X[None]
    if W.ndim == 2:
        W = W[None]
    batch, M, K = X.shape
    if W.shape[0] == 1 and batch > 1:          # one weight matrix shared by every batch element
        W = np.ascontiguousarray(np.broadcast_to(W, (batch,) + W.shape[1:]))
    if W.shape[0] != batch or W.shape[2] != K:
        raise ValueError("shape mismatch between X %s and W %s" % (X.shape, W.shape))
    N = W.shape[1]
    if bias is not None:
        bias = np.ascontiguousarray(bias, dtype=np.float32).reshape(-1)
        if bias.size != (batch * N if bias_per_batch else N):
            raise ValueError("bias has %d elements" % bias.size)
    if scale_vec is not None:
        scale_vec = np.ascontiguousarray(scale_vec, dtype=np.float32).reshape(-1)
        if scale_vec.size != N:
            raise ValueError("scale_vec has %d elements" % scale_vec.size)
    if rows is None:
        nrows, rows_arr = batch * M, None
    else:
        rows_arr = np.ascontiguousarray(rows, dtype=np.int64).reshape(-1)
        nrows = rows_arr.size
    w = out_width(reduce)
    need_y = want_y or reduce == RED_SOFTMAX
    Y = np.empty((nrows, N), dtype=np.float64) if need_y else None
    out = np.empty((nrows, w), dtype=np.float64) if w else None
    prob = _Problem(batch, M, N, K, dtype, act, scale_kind, reduce, float(scale), int(bias_per_batch), 0)
    if residual is not None:
        residual = np.ascontiguousarray(residual)
        if residual.dtype != want or residual.size != batch * M * N:
            raise TypeError("residual must be %s [batch, M, N]" % want.__name__)
        rc = lib().fgr_oracle_rows_residual(ctypes.byref(prob), _ptr(X), _ptr(W), _ptr(bias), _ptr(scale_vec),
                                            _ptr(residual), _ptr(rows_arr), nrows, _ptr(Y), _ptr(out), int(nthreads))
        if rc < 0:
            raise ValueError("fgr_oracle_rows_residual rejected its arguments (code %d)" % rc)
        return Y, out, rc
    rc = lib().fgr_oracle_rows(ctypes.byref(prob), _ptr(X), _ptr(W), _ptr(bias), _ptr(scale_vec), _ptr(rows_arr),
                               nrows, _ptr(Y), _ptr(out), int(nthreads))
    if rc < 0:
        raise ValueError("fgr_oracle_rows rejected its arguments (code %d)" % rc)
    return Y, out, rc


def conv1d_windows(x, taps: int, stride: int = 1):
    """Rows of the 1-D convolution written out as a matrix (no arithmetic, only copies).

    The operator category "convolution" (Section 1; Section 4.1, Datasets; the 1-D case is the paper's
    case study, Section 4.4): for a channels-last input x [batch, L, C] and a filter bank
    w [N, taps, C] (no padding, no dilation, stride s),

        z[b, l, n] = sum_{r = 0 .. taps-1} sum_{c = 0 .. C-1} x[b, l s + r, c] * w[n, r, c],   l = 0 .. (L - taps) // s,

    which is the product of the window matrix  A[b, l, r * C + c] = x[b, l s + r, c]  with  w  viewed as
    [N, taps * C].  This returns A [batch, (L - taps) // s + 1, taps * C]; ``run`` on (A, w) is then the
    definition of the fused convolution + epilogue + reduction over the output channels.
    """
    x = np.ascontiguousarray(x)
    if x.ndim == 2:
        x = x[None]
    batch, L, C = x.shape
    if taps < 1 or taps > L or stride < 1:
        raise ValueError("taps must be in 1..L and stride >= 1")
    Lo = (L - taps) // stride + 1
    A = np.empty((batch, Lo, taps * C), dtype=x.dtype)
    for b in range(batch):
        for l in range(Lo):
            for r in range(taps):
                A[b, l, r * C:(r + 1) * C] = x[b, l * stride + r, :]
    return A


def conv2d_windows(x, R: int, S: int):
    """Rows of the 2-D convolution written out as a matrix (no arithmetic, only copies).

    The operator category "convolution" (Section 1; Section 4.1, Datasets) in its image form: for a
    channels-last input x [batch, H, Wd, C] and a filter bank w [N, R, S, C] (no padding, stride 1, no dilation),

        z[b, p, q, n] = sum_{r < R} sum_{s < S} sum_{c < C} x[b, p + r, q + s, c] * w[n, r, s, c],
        p = 0 .. H - R,  q = 0 .. Wd - S,

    which is the product of the window matrix  A[b, p Q + q, (r S + s) C + c] = x[b, p + r, q + s, c]
    (Q = Wd - S + 1) with  w  viewed as [N, R * S * C].  Returns A [batch, P * Q, R * S * C]; ``run`` on (A, w)
    is then the definition of the fused convolution + epilogue + reduction over the output channels.
    """
    x = np.ascontiguousarray(x)
    if x.ndim == 3:
        x = x[None]
    batch, H, Wd, C = x.shape
    if R < 1 or R > H or S < 1 or S > Wd:
        raise ValueError("the filter must fit inside the image")
    P, Q = H - R + 1, Wd - S + 1
    A = np.empty((batch, P * Q, R * S * C), dtype=x.dtype)
    for b in range(batch):
        for pp in range(P):
            for q in range(Q):
                for r in range(R):
                    for t in range(S):
                        k = (r * S + t) * C
                        A[b, pp * Q + q, k:k + C] = x[b, pp + r, q + t, :]
    return A


def run_problem(p, rows=None, want_y=True, nthreads=0):
    """``run`` on an object carrying X, W, bias, scale_vec and the descriptor fields as attributes.
    With ``p.conv_taps > 1``, ``p.X`` is the channels-last input [batch, L, C] of a 1-D convolution and
    ``p.W`` its filters [batch, N, taps * C]."""
    if getattr(p, "conv_rows", 0) > 1:
        # rows are then indexed over the convolution's own outputs, [batch, P, Q] flattened (no image row pitch)
        return run(conv2d_windows(p.X, p.conv_rows, max(p.conv_taps, 1)), p.W, p.bias, p.scale_vec, dtype=p.dtype, act=p.act,
                   scale_kind=p.scale_kind, reduce=p.reduce, scale=p.scale, bias_per_batch=p.bias_per_batch,
                   rows=rows, want_y=want_y, nthreads=nthreads, residual=getattr(p, "residual", None))
    if getattr(p, "conv_taps", 0) > 1:
        return run(conv1d_windows(p.X, p.conv_taps, getattr(p, "conv_stride", 1) or 1), p.W, p.bias, p.scale_vec, dtype=p.dtype, act=p.act,
                   scale_kind=p.scale_kind, reduce=p.reduce, scale=p.scale, bias_per_batch=p.bias_per_batch,
                   rows=rows, want_y=want_y, nthreads=nthreads, residual=getattr(p, "residual", None))
    return run(p.X, p.W, p.bias, p.scale_vec, dtype=p.dtype, act=p.act, scale_kind=p.scale_kind,
               reduce=p.reduce, scale=p.scale, bias_per_batch=p.bias_per_batch, rows=rows, want_y=want_y,
               nthreads=nthreads, residual=getattr(p, "residual", None))


def reduce_rows(A, *, dtype, kind):
    """Reduction over the last dimension of A [M, N] (fp32 values or uint16 bf16 bit patterns; any
    row stride).  Returns ``(P, out)``: P fp64 [M, N] for SOFTMAX else None; out fp64 [M] (LSE, MAX,
    SUM), [M, 2] (MAXSUM, MAX_SUMEXP) or None (SOFTMAX)."""
    want = np.float32 if dtype == F32 else np.uint16
    if A.dtype != want or A.ndim != 2 or A.strides[1] != A.itemsize:
        raise TypeError("A must be a 2-D %s array with contiguous rows" % want.__name__)
    M, N = A.shape
    lda = A.strides[0] // A.itemsize
    w = {RED_LSE: 1, RED_SOFTMAX: 0, RED_MAXSUM: 2, RED_MAX_SUMEXP: 2, RED_MAX: 1, RED_SUM: 1, RED_MEANVAR: 2}[kind]
    P = np.empty((M, N), np.float64) if kind == RED_SOFTMAX else None
    out = np.empty((M, w) if w == 2 else (M,), np.float64) if w else None
    rc = lib().fgr_oracle_reduce_rows(M, N, dtype, kind, A.ctypes.data_as(ctypes.c_void_p), lda, _ptr(P), _ptr(out))
    if rc < 0:
        raise ValueError("fgr_oracle_reduce_rows rejected its arguments (code %d)" % rc)
    return P, out
