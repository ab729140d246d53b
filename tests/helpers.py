"""Small numpy-only helpers for the tests: tiny random problems and brute-force definitions.

Nothing here calls the oracle or the CUDA library; these are the independent pins."""
import numpy as np


def tiny_problem(rng, n, d, K, density=0.5, values="normal"):
    """Random sparse matrix as CSR (fp32 values), labels, and fp32-representable parameters."""
    mask = rng.random((n, d)) < density
    X = np.where(mask, rng.standard_normal((n, d)), 0.0).astype(np.float32)
    if values == "ones":
        X = mask.astype(np.float32)
    indptr = np.zeros(n + 1, np.int64)
    idx, val = [], []
    for i in range(n):
        cols = np.nonzero(mask[i])[0]
        idx.extend(cols.tolist())
        val.extend(X[i, cols].tolist())
        indptr[i + 1] = len(idx)
    indices = np.asarray(idx, np.int32)
    vals = np.asarray(val, np.float32)
    w0 = float(np.float32(rng.standard_normal() * 0.3))
    w = (rng.standard_normal(d) * 0.3).astype(np.float32).astype(np.float64)
    V = (rng.standard_normal((d, K)) * 0.3).astype(np.float32).astype(np.float64)
    return X.astype(np.float64), mask, indptr, indices, vals, w0, w, V


def fm_pairwise(X, mask, w0, w, V):
    """eq. (fm_model) literally: w0 + sum_j w_j x_j + sum_{j<j'} <v_j,v_j'> x_j x_j'  (O(K nnz^2))."""
    n, d = X.shape
    out = np.zeros(n)
    for i in range(n):
        cols = np.nonzero(mask[i])[0]
        f = w0
        for j in cols:
            f += w[j] * X[i, j]
        for a in range(len(cols)):
            for b in range(a + 1, len(cols)):
                j, jp = cols[a], cols[b]
                f += float(np.dot(V[j], V[jp])) * X[i, j] * X[i, jp]
        out[i] = f
    return out


def loss_np(loss, f, y):
    if loss == 0:
        return 0.5 * (f - y) ** 2
    return np.logaddexp(0.0, -y * f)


def objective_np(X, mask, y, loss, w0, w, V, lam_w, lam_v):
    f = fm_pairwise(X, mask, w0, w, V)
    return loss_np(loss, f, y).mean() + 0.5 * lam_w * np.sum(w * w) + 0.5 * lam_v * np.sum(V * V)


def read_golden(name):
    from pathlib import Path
    rows = []
    for line in (Path(__file__).parent / "golden" / name).read_text().splitlines():
        line = line.strip()
        if line and not line.startswith("#"):
            rows.append(line.split())
    return rows
