"""ctypes binding of the fgr C ABI (include/fgr.h): same names, argument marshalling only.

Every step of the operator runs in the CUDA library; nothing here computes.  There is no CPU
fallback: if ``libfgr.so`` is missing or does not load, importing a symbol raises.
"""
from __future__ import annotations

import ctypes
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libfgr.so")

FGR_OK, FGR_ERR_INVALID_ARG, FGR_ERR_UNSUPPORTED, FGR_ERR_WORKSPACE = 0, 1, 2, 3
FGR_ERR_CUDA, FGR_ERR_DEVICE_TIMEOUT, FGR_ERR_ARCH = 4, 5, 6
FGR_F32, FGR_BF16 = 0, 1
FGR_ACT_NONE, FGR_ACT_RELU, FGR_ACT_GELU_TANH, FGR_ACT_SIGMOID, FGR_ACT_TANH, FGR_ACT_SILU = 0, 1, 2, 3, 4, 5
FGR_SCALE_NONE, FGR_SCALE_SCALAR, FGR_SCALE_PER_COLUMN = 0, 1, 2
FGR_RED_LSE, FGR_RED_SOFTMAX, FGR_RED_MAXSUM, FGR_RED_MAX_SUMEXP = 0, 1, 2, 3
FGR_RED_MEANVAR = 6
FGR_REDUCE_MAX, FGR_REDUCE_SUM = 4, 5
FGR_PATH_AUTO, FGR_PATH_SIMT, FGR_PATH_UMMA_TILED, FGR_PATH_UMMA_STREAM_W, FGR_PATH_SIMT_GEMV = 0, 1, 2, 3, 4
FGR_PATH_UMMA_TF32X3 = 5

FGR_STATIC_SCRATCH_BYTES = 4 << 20

EXPORTS = ("fgr_plan", "fgr_create", "fgr_workspace_bytes", "fgr_get_plan", "fgr_run", "fgr_run_host", "fgr_run_static", "fgr_reduce_rows", "fgr_combine_shards", "fgr_set_residual",
           "fgr_get_status", "fgr_profile_enable", "fgr_profile_read", "fgr_profile_empty_launches", "fgr_destroy", "fgr_status_string", "fgr_path_name")


class fgr_desc(ctypes.Structure):
    _fields_ = [("struct_bytes", ctypes.c_uint32),
                ("batch", ctypes.c_int32), ("M", ctypes.c_int32), ("N", ctypes.c_int32), ("K", ctypes.c_int32),
                ("dtype", ctypes.c_int32), ("act", ctypes.c_int32), ("scale_kind", ctypes.c_int32),
                ("reduce", ctypes.c_int32), ("scale", ctypes.c_float), ("write_y", ctypes.c_int32),
                ("ldx", ctypes.c_int64), ("ldw", ctypes.c_int64), ("ldy", ctypes.c_int64),
                ("bsx", ctypes.c_int64), ("bsw", ctypes.c_int64), ("bsy", ctypes.c_int64),
                ("bias_per_batch", ctypes.c_int32), ("device", ctypes.c_int32),
                ("force_path", ctypes.c_int32), ("force_tile_n", ctypes.c_int32),
                ("force_cta_pair", ctypes.c_int32), ("force_ksub", ctypes.c_int32),
                ("conv_taps", ctypes.c_int32), ("w_shared", ctypes.c_int32),
                ("conv_rows", ctypes.c_int32), ("conv_width", ctypes.c_int32)]


class fgr_reduce_desc(ctypes.Structure):
    _fields_ = [("struct_bytes", ctypes.c_uint32), ("M", ctypes.c_int32), ("N", ctypes.c_int32),
                ("dtype", ctypes.c_int32), ("reduce", ctypes.c_int32), ("device", ctypes.c_int32),
                ("lda", ctypes.c_int64), ("ldp", ctypes.c_int64)]


class fgr_shard_desc(ctypes.Structure):
    _fields_ = [("struct_bytes", ctypes.c_uint32), ("shards", ctypes.c_int32), ("reduce", ctypes.c_int32),
                ("dtype", ctypes.c_int32), ("shard", ctypes.c_int32), ("n_local", ctypes.c_int32),
                ("device", ctypes.c_int32), ("n_total", ctypes.c_int32), ("rows", ctypes.c_int64),
                ("ldp", ctypes.c_int64)]


class fgr_plan_info(ctypes.Structure):
    _fields_ = [("path", ctypes.c_int32), ("tile_m", ctypes.c_int32), ("tile_n", ctypes.c_int32),
                ("stages", ctypes.c_int32), ("parts_per_row", ctypes.c_int32), ("grid", ctypes.c_int32),
                ("launches", ctypes.c_int32), ("smem_bytes", ctypes.c_int32), ("cta_pair", ctypes.c_int32),
                ("ksub", ctypes.c_int32), ("num_tiles", ctypes.c_int64),
                ("workspace_bytes", ctypes.c_uint64), ("flop", ctypes.c_double), ("min_bytes", ctypes.c_double)]

    def as_dict(self):
        return {k: getattr(self, k) for k, _ in self._fields_}


class FgrError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s: %s (status %d)" % (where, fgr_status_string(status), status))


_lib = None


def lib() -> ctypes.CDLL:
    """Loads libfgr.so (built in-tree by ``paper_2511_06345_b200.build``); raises if it is absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("libfgr.so is not built (run `python -m paper_2511_06345_b200.build`); "
                               "there is no fallback path")
        L = ctypes.CDLL(LIB_PATH)
        vp, i = ctypes.c_void_p, ctypes.c_int
        L.fgr_plan.argtypes, L.fgr_plan.restype = [ctypes.POINTER(fgr_desc), i, ctypes.POINTER(fgr_plan_info)], i
        L.fgr_create.argtypes, L.fgr_create.restype = [ctypes.POINTER(fgr_desc), ctypes.POINTER(vp)], i
        L.fgr_workspace_bytes.argtypes, L.fgr_workspace_bytes.restype = [vp], ctypes.c_size_t
        L.fgr_get_plan.argtypes, L.fgr_get_plan.restype = [vp, ctypes.POINTER(fgr_plan_info)], i
        L.fgr_run.argtypes, L.fgr_run.restype = [vp] * 8 + [ctypes.c_size_t, vp], i
        L.fgr_run_host.argtypes, L.fgr_run_host.restype = [vp] * 7, i
        L.fgr_run_static.argtypes, L.fgr_run_static.restype = [ctypes.POINTER(fgr_desc)] + [vp] * 7, i
        L.fgr_reduce_rows.argtypes, L.fgr_reduce_rows.restype = [ctypes.POINTER(fgr_reduce_desc)] + [vp] * 4, i
        L.fgr_combine_shards.argtypes, L.fgr_combine_shards.restype = [ctypes.POINTER(fgr_shard_desc)] + [vp] * 4, i
        L.fgr_set_residual.argtypes, L.fgr_set_residual.restype = [vp, vp, ctypes.c_int64, ctypes.c_int64], i
        L.fgr_get_status.argtypes, L.fgr_get_status.restype = [vp], i
        L.fgr_profile_enable.argtypes, L.fgr_profile_enable.restype = [vp, i], i
        L.fgr_profile_read.argtypes, L.fgr_profile_read.restype = [vp, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(i)], i
        L.fgr_profile_empty_launches.argtypes, L.fgr_profile_empty_launches.restype = [i, i, vp], i
        L.fgr_destroy.argtypes, L.fgr_destroy.restype = [vp], i
        L.fgr_status_string.argtypes, L.fgr_status_string.restype = [i], ctypes.c_char_p
        L.fgr_path_name.argtypes, L.fgr_path_name.restype = [i], ctypes.c_char_p
        _lib = L
    return _lib


def make_desc(batch, M, N, K, dtype, act, scale_kind, reduce, *, scale=1.0, write_y=0, ldx=0, ldw=0, ldy=0,
              bsx=0, bsw=0, bsy=0, bias_per_batch=0, device=0, force_path=FGR_PATH_AUTO, force_tile_n=0, force_cta_pair=0, force_ksub=0,
              conv_taps=0, w_shared=0, conv_rows=0, conv_width=0) -> fgr_desc:
    return fgr_desc(ctypes.sizeof(fgr_desc), batch, M, N, K, dtype, act, scale_kind, reduce, scale, write_y,
                    ldx, ldw, ldy, bsx, bsw, bsy, bias_per_batch, device, force_path, force_tile_n, force_cta_pair, force_ksub, conv_taps, w_shared,
                    conv_rows, conv_width)


def fgr_status_string(status: int) -> str:
    return lib().fgr_status_string(int(status)).decode()


def fgr_path_name(path: int) -> str:
    return lib().fgr_path_name(int(path)).decode()


def fgr_plan(desc: fgr_desc, num_sms: int = 0) -> fgr_plan_info:
    info = fgr_plan_info()
    rc = lib().fgr_plan(ctypes.byref(desc), int(num_sms), ctypes.byref(info))
    if rc != FGR_OK:
        raise FgrError(rc, "fgr_plan")
    return info


def fgr_create(desc: fgr_desc) -> ctypes.c_void_p:
    h = ctypes.c_void_p()
    rc = lib().fgr_create(ctypes.byref(desc), ctypes.byref(h))
    if rc != FGR_OK:
        raise FgrError(rc, "fgr_create")
    return h


def fgr_workspace_bytes(h) -> int:
    return int(lib().fgr_workspace_bytes(h))


def fgr_get_plan(h) -> fgr_plan_info:
    info = fgr_plan_info()
    rc = lib().fgr_get_plan(h, ctypes.byref(info))
    if rc != FGR_OK:
        raise FgrError(rc, "fgr_get_plan")
    return info


def _addr(x):
    """None -> NULL; int -> that address; anything with data_ptr() (a torch tensor) -> its address."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    return x.data_ptr()


def fgr_run(h, X, W, bias, scale_vec, Y, out, workspace, workspace_bytes: int, stream=None, check=True) -> int:
    """Device pointers (ints or tensors).  ``stream``: a raw cudaStream_t value (int) or None."""
    rc = lib().fgr_run(h, _addr(X), _addr(W), _addr(bias), _addr(scale_vec), _addr(Y), _addr(out),
                       _addr(workspace), int(workspace_bytes), stream)
    if check and rc != FGR_OK:
        raise FgrError(rc, "fgr_run")
    return rc


def fgr_run_host(h, X, W, bias, scale_vec, Y, out, check=True) -> int:
    """Host pointers (ints, or CPU tensors / anything with data_ptr())."""
    rc = lib().fgr_run_host(h, _addr(X), _addr(W), _addr(bias), _addr(scale_vec), _addr(Y), _addr(out))
    if check and rc != FGR_OK:
        raise FgrError(rc, "fgr_run_host")
    return rc


def fgr_run_static(desc: fgr_desc, X, W, bias, scale_vec, Y, out, stream=None, check=True) -> int:
    """The operator without a handle or workspace, for callers that cannot allocate device memory:
    the scratch is a fixed array inside the library (see include/fgr.h for the size limit and the
    sharing rules).  Device pointers (ints or tensors); ``stream`` a raw cudaStream_t value or None."""
    rc = lib().fgr_run_static(ctypes.byref(desc), _addr(X), _addr(W), _addr(bias), _addr(scale_vec), _addr(Y),
                              _addr(out), stream)
    if check and rc != FGR_OK:
        raise FgrError(rc, "fgr_run_static")
    return rc


def fgr_reduce_rows(M, N, dtype, reduce, A, P, out, *, lda=0, ldp=0, device=0, stream=None, check=True) -> int:
    """Stand-alone reduction over the rows of A [M, N] (device pointers: ints or tensors)."""
    d = fgr_reduce_desc(ctypes.sizeof(fgr_reduce_desc), M, N, dtype, reduce, device, lda, ldp)
    rc = lib().fgr_reduce_rows(ctypes.byref(d), _addr(A), _addr(P), _addr(out), stream)
    if check and rc != FGR_OK:
        raise FgrError(rc, "fgr_reduce_rows")
    return rc


def fgr_combine_shards(rows, shards, reduce, pairs, out, P_local=None, *, dtype=FGR_BF16, shard=0, n_local=0, ldp=0,
                       device=0, stream=None, check=True, n_total=0) -> int:
    """Merges the all-gathered per-shard row statistics ``pairs`` [shards, rows, 2] of an N-sharded
    operator (device pointers: ints or tensors); softmax also rescales the local slice ``P_local``."""
    d = fgr_shard_desc(ctypes.sizeof(fgr_shard_desc), shards, reduce, dtype, shard, n_local, device, n_total, rows, ldp)
    rc = lib().fgr_combine_shards(ctypes.byref(d), _addr(pairs), _addr(out), _addr(P_local), stream)
    if check and rc != FGR_OK:
        raise FgrError(rc, "fgr_combine_shards")
    return rc


def fgr_set_residual(h, R, ldr: int = 0, bsr: int = 0, check=True) -> int:
    """Sets (or with ``R=None`` removes) the residual tensor added after activation and scale (a device pointer or tensor)."""
    rc = lib().fgr_set_residual(h, _addr(R), int(ldr), int(bsr))
    if check and rc != FGR_OK:
        raise FgrError(rc, "fgr_set_residual")
    return rc


def fgr_get_status(h) -> int:
    return int(lib().fgr_get_status(h))


def fgr_profile_enable(h, enable: bool) -> int:
    return int(lib().fgr_profile_enable(h, int(bool(enable))))


def fgr_profile_read(h):
    """Returns (summed main-kernel milliseconds, runs covered)."""
    ms, n = ctypes.c_double(), ctypes.c_int()
    rc = lib().fgr_profile_read(h, ctypes.byref(ms), ctypes.byref(n))
    if rc != FGR_OK:
        raise FgrError(rc, "fgr_profile_read")
    return ms.value, n.value


def fgr_profile_empty_launches(n: int, device: int = 0, stream=None) -> int:
    """Enqueues n launches of a do-nothing kernel (the caller times them: the launch-latency floor)."""
    rc = int(lib().fgr_profile_empty_launches(int(n), int(device), stream))
    if rc != FGR_OK:
        raise FgrError(rc, "fgr_profile_empty_launches")
    return rc


def fgr_destroy(h) -> int:
    return int(lib().fgr_destroy(h))
