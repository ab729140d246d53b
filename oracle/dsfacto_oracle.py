"""ctypes front end of the CPU oracle (oracle/dsfacto_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by tests/, the smoke check and the bench's CPU-baseline leg.
State is kept in fp64 numpy arrays; see the C file for the passages of the paper each routine
follows and for the readings taken where the paper is garbled."""
from __future__ import annotations

import ctypes

import numpy as np

from .build_oracle import build_oracle

SQUARED, LOGISTIC = 0, 1

_lib = None


def lib():
    global _lib
    if _lib is None:
        L = ctypes.CDLL(str(build_oracle()))
        L.oracle_init_value.restype = ctypes.c_double
        L.oracle_init_value.argtypes = [ctypes.c_uint64, ctypes.c_uint64]
        L.oracle_splitmix64_at.restype = ctypes.c_uint64
        L.oracle_splitmix64_at.argtypes = [ctypes.c_uint64, ctypes.c_uint64]
        L.oracle_bucket.restype = ctypes.c_int
        L.oracle_column_epoch.restype = ctypes.c_int64
        _lib = L
    return _lib


def _p(a):
    return ctypes.c_void_p(a.ctypes.data)


def _i64(v):
    return ctypes.c_int64(int(v))


def _i32(v):
    return ctypes.c_int32(int(v))


def _f64(v):
    return ctypes.c_double(float(v))


def init_params(d, K, seed):
    """Algorithm 1 initialisation: returns (w0, w[d], V[d,K]) in fp64 (values fp32-representable)."""
    w0 = ctypes.c_double(0.0)
    w = np.empty(d, np.float64)
    V = np.empty((d, K), np.float64)
    lib().oracle_init_params(_i32(d), _i32(K), ctypes.c_uint64(seed), ctypes.byref(w0), _p(w), _p(V))
    return w0.value, w, V


def bucket(n, d, p, indptr, indices, values):
    """Tile lists in canonical order (round, row block, column, row): tile_ptr, rows, cols, vals."""
    nnz = int(indptr[-1])
    tile_ptr = np.zeros(p * p + 1, np.int64)
    rows = np.empty(nnz, np.int32)
    cols = np.empty(nnz, np.int32)
    vals = np.empty(nnz, np.float32)
    rc = lib().oracle_bucket(_i64(n), _i32(d), _i32(p), _p(indptr), _p(indices), _p(values),
                             _p(tile_ptr), _p(rows), _p(cols), _p(vals))
    if rc != 0:
        raise MemoryError("oracle_bucket")
    return tile_ptr, rows, cols, vals


def score(indptr, indices, values, w0, w, V):
    m = len(indptr) - 1
    out = np.empty(m, np.float64)
    lib().oracle_score(_i64(m), _i32(V.shape[1]), _p(indptr), _p(indices), _p(values), _f64(w0), _p(w),
                       _p(V), _p(out))
    return out


def evaluate(loss, indptr, indices, values, y, w0, w, V):
    """Held-out mean loss and RMSE (squared loss) or accuracy (logistic loss) of the scores."""
    indptr = np.ascontiguousarray(indptr, np.int64)
    indices = np.ascontiguousarray(indices, np.int32)
    values = np.ascontiguousarray(values, np.float32)
    y = np.ascontiguousarray(y, np.float32)
    out = np.zeros(2, np.float64)
    lib().oracle_evaluate(_i64(len(indptr) - 1), _i32(V.shape[1]), _i32(loss), _p(indptr), _p(indices), _p(values),
                          _p(y), _f64(w0), _p(w), _p(V), _p(out))
    return float(out[0]), float(out[1])


def column_epoch(wl_n, d, K, p, loss, eta_s, lambda_w, lambda_v, indptr, indices, values, y, w0, w, V, j):
    wj = ctypes.c_double(0.0)
    vj = np.empty(K, np.float64)
    cnt = lib().oracle_column_epoch(_i64(wl_n), _i32(d), _i32(K), _i32(p), _i32(loss), _f64(eta_s),
                                    _f64(lambda_w), _f64(lambda_v), _p(indptr), _p(indices), _p(values),
                                    _p(y), _f64(w0), _p(w), _p(V), _i32(j), ctypes.byref(wj), _p(vj))
    return wj.value, vj, int(cnt)


class Oracle:
    """The whole path, step by step: create -> load_csr (bucket + first refresh) -> epoch ..."""

    def __init__(self, n, d, K, p, loss, lambda_w, lambda_v, eta, seed, literal_step=False):
        self.n, self.d, self.K, self.p, self.loss = int(n), int(d), int(K), int(p), int(loss)
        self.lambda_w, self.lambda_v, self.eta = float(lambda_w), float(lambda_v), float(eta)
        # per-nonzero step: eta / N (the objective is normalised by 1/N); literal_step keeps eta
        self.literal_step = bool(literal_step)
        self.eta_s = self.eta if literal_step else self.eta / max(self.n, 1)
        self.w0, self.w, self.V = init_params(self.d, self.K, seed)
        self.loaded = False

    def load_csr(self, indptr, indices, values, y):
        self.indptr = np.ascontiguousarray(indptr, np.int64)
        self.indices = np.ascontiguousarray(indices, np.int32)
        self.values = np.ascontiguousarray(values, np.float32)
        self.y = np.ascontiguousarray(y, np.float32)
        self.tile_ptr, self.rows, self.cols, self.vals = bucket(self.n, self.d, self.p, self.indptr,
                                                                self.indices, self.values)
        n, K = self.n, self.K
        self.A = np.zeros((n, K), np.float64)
        self.lin = np.zeros(n, np.float64)
        self.q = np.zeros(n, np.float64)
        self.f = np.zeros(n, np.float64)
        self.lossv = np.zeros(n, np.float64)
        self.G = np.zeros(n, np.float64)
        self.out3 = np.zeros(3, np.float64)
        self.refresh()
        self.loaded = True

    def refresh(self):
        lib().oracle_refresh(_i64(self.n), _i32(self.d), _i32(self.K), _i32(self.loss), _f64(self.lambda_w),
                             _f64(self.lambda_v), _p(self.indptr), _p(self.indices), _p(self.values),
                             _p(self.y), _f64(self.w0), _p(self.w), _p(self.V), _p(self.A), _p(self.lin),
                             _p(self.q), _p(self.f), _p(self.lossv), _p(self.G), _p(self.out3))

    def sgd_phase(self):
        lib().oracle_sgd_phase(_i32(self.K), _i32(self.p), _f64(self.eta_s), _f64(self.lambda_w),
                               _f64(self.lambda_v), _p(self.tile_ptr), _p(self.rows), _p(self.cols),
                               _p(self.vals), _p(self.A), _p(self.G), _p(self.w), _p(self.V))

    def epoch(self):
        w0 = ctypes.c_double(self.w0)
        lib().oracle_epoch(_i64(self.n), _i32(self.d), _i32(self.K), _i32(self.p), _i32(self.loss),
                           _f64(self.eta_s), _f64(self.lambda_w), _f64(self.lambda_v), _p(self.indptr),
                           _p(self.indices), _p(self.values), _p(self.y), _p(self.tile_ptr), _p(self.rows),
                           _p(self.cols), _p(self.vals), ctypes.byref(w0), _p(self.w), _p(self.V),
                           _p(self.A), _p(self.lin), _p(self.q), _p(self.f), _p(self.lossv), _p(self.G),
                           _p(self.out3))
        self.w0 = w0.value
        return self.objective

    def epoch_segmented(self, every):
        """One epoch with G, A recomputed after every `every` inner rounds (0: after all p)."""
        w0 = ctypes.c_double(self.w0)
        lib().oracle_epoch_segmented(_i64(self.n), _i32(self.d), _i32(self.K), _i32(self.p), _i32(self.loss),
                                     _i32(every), _f64(self.eta_s), _f64(self.lambda_w), _f64(self.lambda_v),
                                     _p(self.indptr), _p(self.indices), _p(self.values), _p(self.y),
                                     _p(self.tile_ptr), _p(self.rows), _p(self.cols), _p(self.vals),
                                     ctypes.byref(w0), _p(self.w), _p(self.V), _p(self.A), _p(self.lin), _p(self.q),
                                     _p(self.f), _p(self.lossv), _p(self.G), _p(self.out3))
        self.w0 = w0.value
        return self.objective

    @property
    def sum_G(self):
        return float(self.out3[0])

    @property
    def mean_loss(self):
        return float(self.out3[1])

    @property
    def objective(self):
        return float(self.out3[2])

    def predict(self, indptr=None, indices=None, values=None):
        if indptr is None:
            indptr, indices, values = self.indptr, self.indices, self.values
        return score(np.ascontiguousarray(indptr, np.int64), np.ascontiguousarray(indices, np.int32),
                     np.ascontiguousarray(values, np.float32), self.w0, self.w, self.V)

    def evaluate(self, indptr, indices, values, y):
        return evaluate(self.loss, indptr, indices, values, y, self.w0, self.w, self.V)

    def set_eta(self, eta):
        """New learning rate for the following epochs (step-size schedules are the caller's)."""
        self.eta = float(eta)
        self.eta_s = self.eta if self.literal_step else self.eta / max(self.n, 1)
