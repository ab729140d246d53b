"""Seeded synthetic workloads (CSR data + labels + training hyper-parameters).

The arrays come from csrc/workloads_gen.c (counter-based random numbers, so a given (name, seed)
always yields the same bytes regardless of thread count).  This module holds no part of the
training method; it is the one piece of code that both the CUDA library's tests/bench and the CPU
oracle's tests take their inputs from.

Named workloads
  C1  tiny regression            n=2,000      d=100      10/row   K=8   squared   p=4
  C2  dense-ish classification   n=50,000     d=22       13/row   K=16  logistic  p=16
  C3  sparse text-like           n=72,000     d=21,000   26..76   K=32  logistic  p=64
  C4  hashed categorical (CTR)   n=45,000,000 d=2^20     39/row   K=16  logistic  p=512
  C5  wide-factor stress         n=4,000,000  d=2^20     100/row  K=128 squared   p=256
  C4s / C5s  the same generators at sizes a CPU reference finishes in seconds.
"""
from __future__ import annotations

import ctypes
import dataclasses
from typing import Optional

import numpy as np

from . import build as _build

SQUARED, LOGISTIC = 0, 1


class _Spec(ctypes.Structure):
    _fields_ = [
        ("n", ctypes.c_int64), ("d", ctypes.c_int32), ("seed", ctypes.c_uint64),
        ("structure", ctypes.c_int32), ("len_min", ctypes.c_int32), ("len_max", ctypes.c_int32),
        ("n_fields", ctypes.c_int32), ("field_range", ctypes.c_int32), ("zipf_s", ctypes.c_double),
        ("value_kind", ctypes.c_int32), ("label_kind", ctypes.c_int32), ("k_star", ctypes.c_int32),
        ("w_scale", ctypes.c_double), ("v_scale", ctypes.c_double), ("support_frac", ctypes.c_double),
        ("noise", ctypes.c_double), ("flip", ctypes.c_double), ("bias", ctypes.c_double),
    ]


_lib = None


def _gen():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(str(_build.build_workloads()))
        lib.wl_row_pointers.argtypes = [ctypes.POINTER(_Spec), ctypes.c_void_p]
        lib.wl_row_pointers.restype = ctypes.c_int
        lib.wl_fill.argtypes = [ctypes.POINTER(_Spec)] + [ctypes.c_void_p] * 4
        lib.wl_fill.restype = ctypes.c_int
        _lib = lib
    return _lib


UNIFORM, ZIPF, FIELDS = 0, 1, 2
V_NORMAL, V_UNIFORM, V_LOGNORMAL_L2, V_ONES = 0, 1, 2, 3
L_REGRESSION, L_SIGN, L_BERNOULLI, L_SCORE = 0, 1, 2, 3

# data description + training hyper-parameters of every named workload
CONFIGS = {
    "C1": dict(n=2_000, d=100, structure=UNIFORM, len_min=10, len_max=10, value_kind=V_NORMAL,
               label_kind=L_REGRESSION, k_star=4, w_scale=1.0, v_scale=0.5, noise=0.1,
               K=8, loss=SQUARED, p=4, eta=0.01, epochs=10, seed=13941),
    "C2": dict(n=50_000, d=22, structure=UNIFORM, len_min=13, len_max=13, value_kind=V_UNIFORM,
               label_kind=L_SIGN, k_star=8, w_scale=1.0, v_scale=0.5, flip=0.10,
               K=16, loss=LOGISTIC, p=16, eta=4.0, epochs=20, seed=13942),
    "C3": dict(n=72_000, d=21_000, structure=ZIPF, len_min=26, len_max=76, zipf_s=1.1,
               value_kind=V_LOGNORMAL_L2, label_kind=L_SIGN, k_star=8, w_scale=1.0, v_scale=0.5,
               support_frac=0.10, K=32, loss=LOGISTIC, p=64, eta=8.0, epochs=5, seed=13943),
    "C4": dict(n=45_000_000, d=1 << 20, structure=FIELDS, n_fields=39, field_range=26_886, zipf_s=1.2,
               value_kind=V_ONES, label_kind=L_BERNOULLI, k_star=8, w_scale=0.3, v_scale=0.1,
               positive_rate=0.25, K=16, loss=LOGISTIC, p=512, eta=1.0, epochs=1, seed=13944),
    "C5": dict(n=4_000_000, d=1 << 20, structure=ZIPF, len_min=100, len_max=100, zipf_s=1.05,
               value_kind=V_NORMAL, label_kind=L_REGRESSION, k_star=16, w_scale=0.3, v_scale=0.1,
               noise=0.1, K=128, loss=SQUARED, p=256, eta=0.05, epochs=2, seed=13945),
}
# reduced variants: same generators and column structure, fewer rows / tiles
CONFIGS["C4s"] = dict(CONFIGS["C4"], n=200_000, p=32)
CONFIGS["C5s"] = dict(CONFIGS["C5"], n=40_000, d=1 << 17, p=16)


@dataclasses.dataclass
class Workload:
    name: str
    n: int
    d: int
    K: int
    p: int
    loss: int
    eta: float
    lambda_w: float
    lambda_v: float
    epochs: int
    init_seed: int
    indptr: np.ndarray    # int64 [n+1]
    indices: np.ndarray   # int32 [nnz], strictly increasing inside a row
    values: np.ndarray    # float32 [nnz]
    y: np.ndarray         # float32 [n]

    @property
    def nnz(self) -> int:
        return int(self.indptr[-1])


def generate(n, d, seed, structure, len_min=0, len_max=0, n_fields=0, field_range=0, zipf_s=1.0,
             value_kind=V_NORMAL, label_kind=L_REGRESSION, k_star=4, w_scale=1.0, v_scale=0.5,
             support_frac=1.0, noise=0.0, flip=0.0, bias=0.0, empty=np.empty):
    """Raw generator call -> (indptr, indices, values, y).  `empty` allocates the output arrays
    (pass a pinned-memory allocator to get page-locked buffers)."""
    spec = _Spec(n=n, d=d, seed=seed, structure=structure, len_min=len_min, len_max=len_max,
                 n_fields=n_fields, field_range=field_range, zipf_s=zipf_s, value_kind=value_kind,
                 label_kind=label_kind, k_star=k_star, w_scale=w_scale, v_scale=v_scale,
                 support_frac=support_frac, noise=noise, flip=flip, bias=bias)
    lib = _gen()
    indptr = empty(n + 1, dtype=np.int64)
    if lib.wl_row_pointers(ctypes.byref(spec), indptr.ctypes.data) != 0:
        raise ValueError("invalid workload description")
    nnz = int(indptr[-1])
    indices = empty(max(nnz, 1), dtype=np.int32)[:nnz]
    values = empty(max(nnz, 1), dtype=np.float32)[:nnz]
    y = empty(max(n, 1), dtype=np.float32)[:n]
    rc = lib.wl_fill(ctypes.byref(spec), indptr.ctypes.data, indices.ctypes.data, values.ctypes.data,
                     y.ctypes.data)
    if rc != 0:
        raise MemoryError("workload generator failed (%d)" % rc)
    return indptr, indices, values, y


def _bias_for_rate(cfg: dict, rate: float) -> float:
    """Intercept b with mean(sigmoid(score + b)) = rate on the first <=1M rows (bisection)."""
    m = min(cfg["n"], 1_000_000)
    keys = ("d", "seed", "structure", "len_min", "len_max", "n_fields", "field_range", "zipf_s",
            "value_kind", "k_star", "w_scale", "v_scale", "support_frac")
    kw = {k: cfg[k] for k in keys if k in cfg}
    score = generate(n=m, label_kind=L_SCORE, **kw)[3].astype(np.float64)
    lo, hi = -30.0, 30.0
    for _ in range(60):
        mid = 0.5 * (lo + hi)
        if np.mean(1.0 / (1.0 + np.exp(-(score + mid)))) < rate:
            lo = mid
        else:
            hi = mid
    return 0.5 * (lo + hi)


def make(name: str, n: Optional[int] = None, p: Optional[int] = None, empty=np.empty) -> Workload:
    """Builds the named workload; `n` / `p` override the row count / tile grid (for scaled runs)."""
    cfg = dict(CONFIGS[name])
    if n is not None:
        cfg["n"] = int(n)
    if p is not None:
        cfg["p"] = int(p)
    if "positive_rate" in cfg:
        cfg["bias"] = _bias_for_rate(cfg, cfg["positive_rate"])
    keys = ("n", "d", "seed", "structure", "len_min", "len_max", "n_fields", "field_range", "zipf_s",
            "value_kind", "label_kind", "k_star", "w_scale", "v_scale", "support_frac", "noise", "flip",
            "bias")
    indptr, indices, values, y = generate(empty=empty, **{k: cfg[k] for k in keys if k in cfg})
    return Workload(name=name, n=cfg["n"], d=cfg["d"], K=cfg["K"], p=cfg["p"], loss=cfg["loss"],
                    eta=cfg["eta"], lambda_w=1e-3, lambda_v=1e-3, epochs=cfg["epochs"], init_seed=2004,
                    indptr=indptr, indices=indices, values=values, y=y)
