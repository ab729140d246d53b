"""ctypes binding of the CUDA C-ABI library (include/dsfacto.h).

Argument marshalling only: every step of the path runs inside libdsfacto.so.  There is no CPU
fallback: if the library is missing or cannot be built, importing symbols raises; if no CUDA
device is usable, dsfacto_create returns DSFACTO_ERR_CUDA and `DSFacto(...)` raises."""
from __future__ import annotations

import ctypes
from typing import Optional

import numpy as np

from . import build as _build

SQUARED, LOGISTIC = 0, 1
OK, ERR_INVALID_ARG, ERR_INVALID_CSR, ERR_NO_DATA, ERR_OOM, ERR_CUDA, ERR_DIVERGED = 0, -1, -2, -3, -4, -5, -6

_c_i64, _c_i32, _c_f32, _c_u64, _vp = ctypes.c_int64, ctypes.c_int32, ctypes.c_float, ctypes.c_uint64, ctypes.c_void_p

# name -> (restype, argtypes); one entry per declaration in include/dsfacto.h
SIGNATURES = {
    "dsfacto_create": (ctypes.c_int, [ctypes.POINTER(_vp), _c_i64, _c_i32, _c_i32, _c_i32, _c_i32, _c_f32, _c_f32,
                                      _c_f32, _c_u64]),
    "dsfacto_load_csr": (ctypes.c_int, [_vp, _vp, _vp, _vp, _vp]),
    "dsfacto_epoch": (ctypes.c_int, [_vp]),
    "dsfacto_predict": (ctypes.c_int, [_vp, _c_i64, _vp, _vp, _vp, _vp]),
    "dsfacto_evaluate": (ctypes.c_int, [_vp, _c_i64, _vp, _vp, _vp, _vp, ctypes.POINTER(ctypes.c_double),
                                        ctypes.POINTER(ctypes.c_double)]),
    "dsfacto_set_eta": (ctypes.c_int, [_vp, _c_f32]),
    "dsfacto_set_refresh_every": (ctypes.c_int, [_vp, _c_i32]),
    "dsfacto_objective": (ctypes.c_int, [_vp, ctypes.POINTER(ctypes.c_double)]),
    "dsfacto_get_params": (ctypes.c_int, [_vp, _vp, _vp, _vp]),
    "dsfacto_set_params": (ctypes.c_int, [_vp, _vp, _vp, _vp]),
    "dsfacto_destroy": (None, [_vp]),
    "dsfacto_get_tiles": (ctypes.c_int, [_vp, _vp, _vp, _vp, _vp]),
    "dsfacto_bucket_host": (ctypes.c_int, [_c_i64, _c_i32, _c_i32, _vp, _vp, _vp, _vp, _vp, _vp, _vp]),
    "dsfacto_get_aux": (ctypes.c_int, [_vp, _vp, _vp]),
    "dsfacto_get_stats": (ctypes.c_int, [_vp, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_double)]),
    "dsfacto_set_stream": (ctypes.c_int, [_vp, _vp]),
    "dsfacto_last_epoch_ms": (ctypes.c_int, [_vp, ctypes.POINTER(ctypes.c_float)]),
    "dsfacto_debug_set": (ctypes.c_int, [_vp, _c_i32, _c_i64]),
    "dsfacto_create_shard": (ctypes.c_int, [ctypes.POINTER(_vp), _c_i64, _c_i32, _c_i32, _c_i32, _c_i32, _c_f32, _c_f32,
                                            _c_f32, _c_u64, _c_i32, _c_i32]),
    "dsfacto_shard_columns": (ctypes.c_int, [_vp, ctypes.POINTER(_c_i32), ctypes.POINTER(_c_i32)]),
    "dsfacto_shard_partial_count": (ctypes.c_int, [_vp, ctypes.POINTER(_c_i64)]),
    "dsfacto_shard_epoch_begin": (ctypes.c_int, [_vp]),
    "dsfacto_shard_partial": (ctypes.c_int, [_vp, _vp, _c_i64]),
    "dsfacto_shard_epoch_end": (ctypes.c_int, [_vp, _vp, _c_i64, ctypes.POINTER(ctypes.c_double)]),
    "dsfacto_bucket_host_shard": (ctypes.c_int, [_c_i64, _c_i32, _c_i32, _c_i32, _c_i32, _vp, _vp, _vp,
                                                 ctypes.POINTER(_c_i64), _vp, _vp, _vp, _vp]),
    "dsfacto_launch_count": (ctypes.c_int, [_vp, ctypes.POINTER(_c_i64)]),
    "dsfacto_last_load": (ctypes.c_int, [_vp, ctypes.POINTER(_c_i64)]),
    "dsfacto_last_error": (ctypes.c_char_p, [_vp]),
    "dsfacto_strerror": (ctypes.c_char_p, [ctypes.c_int]),
    "dsfacto_score_loss_noalloc": (ctypes.c_int, [_c_i64, _c_i32, _c_i32, _c_i32, _vp, _vp, _vp, _vp, _c_f32, _vp, _vp,
                                                  _vp, _vp, _vp]),
}

_lib = None


def _load(path) -> ctypes.CDLL:
    L = ctypes.CDLL(str(path))
    for name, (res, args) in SIGNATURES.items():
        fn = getattr(L, name)
        fn.restype, fn.argtypes = res, args
    return L


def lib() -> ctypes.CDLL:
    """Loads (building first if the sources are newer) libdsfacto.so; raises if that fails."""
    global _lib
    if _lib is None:
        _lib = _load(_build.build_cuda())
    return _lib


class use_debug_library:
    """Context manager: inside it every call of this module goes to libdsfacto_debug.so, the same sources
    built with -DDSFACTO_DEBUG (index checks in the stratum SGD kernel that report instead of trapping)."""

    def __enter__(self):
        global _lib
        self._saved = lib()
        _lib = _load(_build.build_cuda(debug=True))
        return _lib

    def __exit__(self, *exc):
        global _lib
        _lib = self._saved


class DSFactoError(RuntimeError):
    def __init__(self, status: int, where: str, detail: str = ""):
        self.status = status
        msg = lib().dsfacto_strerror(status).decode()
        super().__init__("%s: %s (%d)%s" % (where, msg, status, (": " + detail) if detail else ""))


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else ctypes.c_void_p(a.ctypes.data)


# ---- the C calls under their own names (thin wrappers: numpy arrays in, status out) ----
def dsfacto_create(n, d, K, p, loss, lambda_w, lambda_v, eta, seed):
    h = _vp()
    rc = lib().dsfacto_create(ctypes.byref(h), n, d, K, p, loss, lambda_w, lambda_v, eta, seed)
    return rc, h


def dsfacto_load_csr(h, indptr, indices, values, y):
    return lib().dsfacto_load_csr(h, _ptr(indptr), _ptr(indices), _ptr(values), _ptr(y))


def dsfacto_epoch(h):
    return lib().dsfacto_epoch(h)


def dsfacto_predict(h, m, indptr, indices, values, out):
    return lib().dsfacto_predict(h, m, _ptr(indptr), _ptr(indices), _ptr(values), _ptr(out))


def dsfacto_evaluate(h, m, indptr, indices, values, y):
    ml, mt = ctypes.c_double(), ctypes.c_double()
    rc = lib().dsfacto_evaluate(h, m, _ptr(indptr), _ptr(indices), _ptr(values), _ptr(y), ctypes.byref(ml),
                                ctypes.byref(mt))
    return rc, ml.value, mt.value


def dsfacto_set_eta(h, eta):
    return lib().dsfacto_set_eta(h, eta)


def dsfacto_set_refresh_every(h, rounds):
    return lib().dsfacto_set_refresh_every(h, rounds)


DEBUG_SPIN_LIMIT, DEBUG_EXTRA_NEED, DEBUG_CHUNK_LEN, DEBUG_COLUMN_ORDER, DEBUG_ROW_MERGE = 0, 1, 2, 3, 4


def dsfacto_debug_set(h, key, value):
    return lib().dsfacto_debug_set(h, key, value)


def dsfacto_objective(h):
    v = ctypes.c_double()
    rc = lib().dsfacto_objective(h, ctypes.byref(v))
    return rc, v.value


def dsfacto_get_params(h, w0, w, V):
    return lib().dsfacto_get_params(h, _ptr(w0), _ptr(w), _ptr(V))


def dsfacto_set_params(h, w0, w, V):
    return lib().dsfacto_set_params(h, _ptr(w0), _ptr(w), _ptr(V))


def dsfacto_destroy(h):
    lib().dsfacto_destroy(h)


def dsfacto_bucket_host(n, d, p, indptr, indices, values):
    """Host tile bucketer alone -> (status, tile_ptr, rows, cols, vals); needs no GPU."""
    nnz = int(indptr[-1])
    tile_ptr = np.zeros(p * p + 1, np.int64)
    rows = np.empty(max(nnz, 1), np.int32)[:nnz]
    cols = np.empty(max(nnz, 1), np.int32)[:nnz]
    vals = np.empty(max(nnz, 1), np.float32)[:nnz]
    rc = lib().dsfacto_bucket_host(n, d, p, _ptr(indptr), _ptr(indices), _ptr(values), _ptr(tile_ptr), _ptr(rows),
                                   _ptr(cols), _ptr(vals))
    return rc, tile_ptr, rows, cols, vals


def dsfacto_bucket_host_shard(n, d, p, shard, nshards, indptr, indices, values):
    """Host tile bucketer of one column shard -> (status, kept, tile_ptr, rows, cols, vals); needs no GPU."""
    nnz = int(indptr[-1])
    tile_ptr = np.zeros(p * p + 1, np.int64)
    rows = np.empty(max(nnz, 1), np.int32)
    cols = np.empty(max(nnz, 1), np.int32)
    vals = np.empty(max(nnz, 1), np.float32)
    kept = _c_i64()
    rc = lib().dsfacto_bucket_host_shard(n, d, p, shard, nshards, _ptr(indptr), _ptr(indices), _ptr(values),
                                         ctypes.byref(kept), _ptr(tile_ptr), _ptr(rows), _ptr(cols), _ptr(vals))
    k = int(kept.value)
    return rc, k, tile_ptr, rows[:k], cols[:k], vals[:k]


def dsfacto_score_loss_noalloc(m, d, K, loss, indptr_dev, indices_dev, values_dev, y_dev, w0, w_dev, V_dev,
                               scores_dev, sums_dev, cuda_stream=0):
    """Allocation-free scoring; every *_dev argument is a raw device address (int)."""
    vp = lambda a: ctypes.c_void_p(int(a))
    return lib().dsfacto_score_loss_noalloc(m, d, K, loss, vp(indptr_dev), vp(indices_dev), vp(values_dev), vp(y_dev),
                                            w0, vp(w_dev), vp(V_dev), vp(scores_dev), vp(sums_dev), vp(cuda_stream))


class DSFacto:
    """Convenience owner of one handle.  Every method is one C call plus array allocation."""

    def __init__(self, n, d, K, p, loss, lambda_w, lambda_v, eta, seed, shard=0, nshards=1):
        self.n, self.d, self.K, self.p = int(n), int(d), int(K), int(p)
        self.shard, self.nshards = int(shard), int(nshards)
        if self.nshards == 1:
            rc, self._h = dsfacto_create(self.n, self.d, self.K, self.p, int(loss), float(lambda_w), float(lambda_v),
                                         float(eta), int(seed))
        else:
            self._h = _vp()
            rc = lib().dsfacto_create_shard(ctypes.byref(self._h), self.n, self.d, self.K, self.p, int(loss),
                                            float(lambda_w), float(lambda_v), float(eta), int(seed), self.shard,
                                            self.nshards)
        if rc != OK:
            self._h = None
            raise DSFactoError(rc, "dsfacto_create")
        self.nnz = 0

    # ---- column shards (see include/dsfacto.h) ----
    def shard_columns(self):
        lo, hi = _c_i32(), _c_i32()
        self._check(lib().dsfacto_shard_columns(self._h, ctypes.byref(lo), ctypes.byref(hi)), "dsfacto_shard_columns")
        return int(lo.value), int(hi.value)

    def shard_partial_count(self) -> int:
        c = _c_i64()
        self._check(lib().dsfacto_shard_partial_count(self._h, ctypes.byref(c)), "dsfacto_shard_partial_count")
        return int(c.value)

    def shard_epoch_begin(self):
        self._check(lib().dsfacto_shard_epoch_begin(self._h), "dsfacto_shard_epoch_begin")

    def shard_partial(self, dst_dev_ptr: int, count: int):
        self._check(lib().dsfacto_shard_partial(self._h, ctypes.c_void_p(dst_dev_ptr), count), "dsfacto_shard_partial")

    def shard_epoch_end(self, summed_dev_ptr: int, count: int):
        sums = (ctypes.c_double * 4)()
        self._check(lib().dsfacto_shard_epoch_end(self._h, ctypes.c_void_p(summed_dev_ptr), count, sums),
                    "dsfacto_shard_epoch_end")
        return [float(x) for x in sums]

    def _check(self, rc, where):
        if rc != OK:
            raise DSFactoError(rc, where, lib().dsfacto_last_error(self._h).decode())

    def close(self):
        if getattr(self, "_h", None):
            dsfacto_destroy(self._h)
            self._h = None

    def __del__(self):
        self.close()

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    def set_stream(self, cuda_stream_ptr: int):
        self._check(lib().dsfacto_set_stream(self._h, ctypes.c_void_p(cuda_stream_ptr)), "dsfacto_set_stream")

    def load_csr(self, indptr, indices, values, y):
        indptr = np.ascontiguousarray(indptr, np.int64)
        indices = np.ascontiguousarray(indices, np.int32)
        values = np.ascontiguousarray(values, np.float32)
        y = np.ascontiguousarray(y, np.float32)
        if indptr.shape != (self.n + 1,) or y.shape != (self.n,):
            raise ValueError("indptr must have n+1 entries and y n entries")
        if indices.shape[0] < indptr[-1] or values.shape[0] < indptr[-1]:
            raise ValueError("indices/values shorter than indptr[-1]")
        self._check(dsfacto_load_csr(self._h, indptr, indices, values, y), "dsfacto_load_csr")
        self.nnz = int(indptr[-1])
        if self.nshards > 1:   # a shard keeps the entries of its own columns only
            lo, hi = self.shard_columns()
            self.nnz = int(np.count_nonzero((indices[: self.nnz] >= lo) & (indices[: self.nnz] < hi)))

    def epoch(self) -> float:
        self._check(dsfacto_epoch(self._h), "dsfacto_epoch")
        return self.objective()

    def objective(self) -> float:
        rc, v = dsfacto_objective(self._h)
        self._check(rc, "dsfacto_objective")
        return v

    def stats(self):
        ml, sg = ctypes.c_double(), ctypes.c_double()
        self._check(lib().dsfacto_get_stats(self._h, ctypes.byref(ml), ctypes.byref(sg)), "dsfacto_get_stats")
        return ml.value, sg.value

    def get_params(self):
        w0 = np.zeros(1, np.float32)
        w = np.empty(self.d, np.float32)
        V = np.empty((self.d, self.K), np.float32)
        self._check(dsfacto_get_params(self._h, w0, w, V), "dsfacto_get_params")
        return float(w0[0]), w, V

    def set_params(self, w0=None, w=None, V=None):
        w0a = None if w0 is None else np.asarray([w0], np.float32)
        wa = None if w is None else np.ascontiguousarray(w, np.float32)
        Va = None if V is None else np.ascontiguousarray(V, np.float32)
        if wa is not None and wa.shape != (self.d,):
            raise ValueError("w must have d entries")
        if Va is not None and Va.shape != (self.d, self.K):
            raise ValueError("V must be d x K")
        self._check(dsfacto_set_params(self._h, w0a, wa, Va), "dsfacto_set_params")

    def predict(self, indptr=None, indices=None, values=None):
        if indptr is None:
            out = np.empty(self.n, np.float32)
            self._check(dsfacto_predict(self._h, self.n, None, None, None, out), "dsfacto_predict")
            return out
        indptr = np.ascontiguousarray(indptr, np.int64)
        indices = np.ascontiguousarray(indices, np.int32)
        values = np.ascontiguousarray(values, np.float32)
        m = indptr.shape[0] - 1
        out = np.empty(max(m, 1), np.float32)[:m]
        self._check(dsfacto_predict(self._h, m, indptr, indices, values, out), "dsfacto_predict")
        return out

    def evaluate(self, indptr, indices, values, y):
        """Held-out (mean loss, RMSE or accuracy) of the rows given as CSR with labels y."""
        indptr = np.ascontiguousarray(indptr, np.int64)
        indices = np.ascontiguousarray(indices, np.int32)
        values = np.ascontiguousarray(values, np.float32)
        y = np.ascontiguousarray(y, np.float32)
        m = indptr.shape[0] - 1
        if y.shape != (m,):
            raise ValueError("y must have one label per row")
        rc, ml, mt = dsfacto_evaluate(self._h, m, indptr, indices, values, y)
        self._check(rc, "dsfacto_evaluate")
        return ml, mt

    def set_eta(self, eta: float):
        self._check(dsfacto_set_eta(self._h, float(eta)), "dsfacto_set_eta")

    def set_refresh_every(self, rounds: int):
        """G, A recomputed after every `rounds` inner rounds (0: once per epoch).  Before load_csr."""
        self._check(dsfacto_set_refresh_every(self._h, int(rounds)), "dsfacto_set_refresh_every")

    def get_tiles(self):
        tile_ptr = np.empty(self.p * self.p + 1, np.int64)
        rows = np.empty(max(self.nnz, 1), np.int32)[: self.nnz]
        cols = np.empty(max(self.nnz, 1), np.int32)[: self.nnz]
        vals = np.empty(max(self.nnz, 1), np.float32)[: self.nnz]
        self._check(lib().dsfacto_get_tiles(self._h, _ptr(tile_ptr), _ptr(rows), _ptr(cols), _ptr(vals)),
                    "dsfacto_get_tiles")
        return tile_ptr, rows, cols, vals

    def get_aux(self):
        A = np.empty((self.n, self.K), np.float32)
        G = np.empty(self.n, np.float32)
        self._check(lib().dsfacto_get_aux(self._h, _ptr(A), _ptr(G)), "dsfacto_get_aux")
        return A, G

    def last_epoch_ms(self):
        ms = (ctypes.c_float * 4)()
        self._check(lib().dsfacto_last_epoch_ms(self._h, ms), "dsfacto_last_epoch_ms")
        return [float(x) for x in ms]

    def debug_set(self, key: int, value: int):
        self._check(dsfacto_debug_set(self._h, int(key), int(value)), "dsfacto_debug_set")

    def last_load(self):
        """(path, bytes host -> device, bytes device -> host) of the last load; path 0 host, 1 host streamed, 2 device."""
        info = (_c_i64 * 3)()
        self._check(lib().dsfacto_last_load(self._h, info), "dsfacto_last_load")
        return int(info[0]), int(info[1]), int(info[2])

    def launch_count(self) -> int:
        v = _c_i64()
        self._check(lib().dsfacto_launch_count(self._h, ctypes.byref(v)), "dsfacto_launch_count")
        return int(v.value)
