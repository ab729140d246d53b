"""Pins for the oracle's schedule and update side: tile bucketing, the stratified order, the
per-nonzero update, and the epoch as a whole.  References are brute force in numpy, closed forms
of the frozen-auxiliary update, finite differences and textbook special cases."""
import numpy as np
import pytest

from oracle import dsfacto_oracle as O
from paper_2004_13940_b200 import workloads as W
from tests.helpers import fm_pairwise, loss_np, tiny_problem


def brute_force_order(n, d, p, indptr, indices):
    """(tile_ptr, permutation of stored entries) by sorting keys (round, row block, column, row)."""
    rows = np.repeat(np.arange(n, dtype=np.int64), np.diff(indptr))
    cols = indices.astype(np.int64)
    rb = rows * p // n
    cb = cols * p // d
    s = (cb - rb) % p
    order = np.lexsort((rows, cols, rb, s))
    tile = (s * p + rb)[order]
    tile_ptr = np.searchsorted(tile, np.arange(p * p + 1), side="left").astype(np.int64)
    return tile_ptr, order, rows, cols, rb, cb, s


@pytest.mark.parametrize("n,d,p,density", [(40, 30, 4, 0.3), (17, 5, 3, 0.7), (9, 3, 5, 0.9), (25, 11, 1, 0.4),
                                           (6, 40, 6, 0.2)])
def test_bucketing_matches_brute_force_sort(n, d, p, density):
    rng = np.random.default_rng(n * 100 + d)
    X, mask, indptr, indices, vals, *_ = tiny_problem(rng, n, d, 2, density)
    tile_ptr, rows, cols, tv = O.bucket(n, d, p, indptr, indices, vals)
    bp, order, r_all, c_all, rb, cb, s = brute_force_order(n, d, p, indptr, indices)
    assert np.array_equal(tile_ptr, bp)
    assert np.array_equal(rows, r_all[order].astype(np.int32))
    assert np.array_equal(cols, c_all[order].astype(np.int32))
    assert np.array_equal(tv.view(np.uint32), vals[order].view(np.uint32))
    assert tile_ptr[-1] == len(indices)                       # every stored entry exactly once
    # Latin square: the p tiles of a round cover every row block and every column block once
    for sr in range(p):
        cbs = sorted(((r + sr) % p) for r in range(p))
        assert cbs == list(range(p))
    for t in range(p * p):
        sr, r = divmod(t, p)
        seg = slice(tile_ptr[t], tile_ptr[t + 1])
        assert np.all(rows[seg].astype(np.int64) * p // n == r)
        assert np.all(cols[seg].astype(np.int64) * p // d == (r + sr) % p)


def test_p1_is_csc_order():
    rng = np.random.default_rng(5)
    n, d = 13, 7
    X, mask, indptr, indices, vals, *_ = tiny_problem(rng, n, d, 2, 0.5)
    tile_ptr, rows, cols, tv = O.bucket(n, d, 1, indptr, indices, vals)
    jj, ii = np.nonzero(mask.T)                               # column-major traversal
    assert np.array_equal(cols, jj.astype(np.int32)) and np.array_equal(rows, ii.astype(np.int32))
    np.testing.assert_array_equal(tv, X[ii, jj].astype(np.float32))


def _setup(seed, n, d, K, p, loss, density=0.5, lam=(1e-2, 2e-2), eta=0.3):
    rng = np.random.default_rng(seed)
    X, mask, indptr, indices, vals, w0, w, V = tiny_problem(rng, n, d, K, density)
    y = (np.where(rng.random(n) < 0.5, 1.0, -1.0) if loss else rng.standard_normal(n)).astype(np.float32)
    o = O.Oracle(n, d, K, p, loss, lam[0], lam[1], eta, seed=3)
    o.w0, o.w[:], o.V[:] = w0, w, V
    o.load_csr(indptr, indices, vals, y)
    return o, X, mask, y.astype(np.float64)


@pytest.mark.parametrize("loss,p", [(O.SQUARED, 3), (O.LOGISTIC, 4), (O.SQUARED, 1)])
def test_sgd_phase_closed_form_per_column(loss, p):
    # With G and A frozen, each update of column j is the affine map
    #   w_j <- (1 - h lw) w_j - h G_i x,   v_j <- (1 - h lv + h G_i x^2) v_j - h G_i x a_i
    # so the end value is the ordered product/sum of those maps over the column's entries, taken in
    # the stratified order (row blocks c, c-1, ... mod p; rows ascending inside a block).
    n, d, K = 31, 8, 3
    o, X, mask, y = _setup(7 + p, n, d, K, p, loss)
    A0, G0, w_start, V_start = o.A.copy(), o.G.copy(), o.w.copy(), o.V.copy()
    o.sgd_phase()
    h, lw, lv = o.eta_s, o.lambda_w, o.lambda_v
    differs = 0
    for j in range(d):
        c = j * p // d
        rows_j = np.nonzero(mask[:, j])[0]
        rnd = (c - rows_j * p // n) % p
        order = rows_j[np.lexsort((rows_j, rnd))]
        for direction, seq in (("fwd", order), ("rev", order[::-1])):
            wj, vj = w_start[j], V_start[j].copy()
            for i in seq:
                x = X[i, j]
                wj = (1 - h * lw) * wj - h * G0[i] * x
                vj = (1 - h * lv + h * G0[i] * x * x) * vj - h * G0[i] * x * A0[i]
            if direction == "fwd":
                assert o.w[j] == pytest.approx(wj, rel=1e-11, abs=1e-14)
                np.testing.assert_allclose(o.V[j], vj, rtol=1e-11, atol=1e-14)
            elif len(seq) > 1:
                differs += int(not np.allclose(o.V[j], vj, rtol=1e-9, atol=0))
    assert differs > 0          # order sensitivity: the reversed sweep is a different result
    assert np.array_equal(o.A, A0) and np.array_equal(o.G, G0)   # auxiliaries stay frozen


@pytest.mark.parametrize("loss", [O.SQUARED, O.LOGISTIC])
def test_epoch_tends_to_gradient_step_of_frequency_weighted_objective(loss):
    # (theta_1 - theta_0)/eta -> -grad of (1/n) sum_i [ l_i + sum_{j in nnz(i)} (lw/2 w_j^2 + lv/2 |v_j|^2) ]
    # as eta -> 0, with the error proportional to eta.  The gradient is a central difference of the
    # brute-force pairwise objective, so signs, the x^2 term, G, a_i and the step scaling are all pinned.
    n, d, K, p = 14, 5, 2, 2
    lam_w, lam_v = 0.05, 0.08
    rng = np.random.default_rng(42 + loss)
    X, mask, indptr, indices, vals, w0, w, V = tiny_problem(rng, n, d, K, 0.6)
    y = (np.where(rng.random(n) < 0.5, 1.0, -1.0) if loss else rng.standard_normal(n)).astype(np.float32)
    yd = y.astype(np.float64)
    cnt = mask.sum(0).astype(np.float64)

    def fw_obj(w0_, w_, V_):
        f = fm_pairwise(X, mask, w0_, w_, V_)
        return (loss_np(loss, f, yd).sum() + 0.5 * lam_w * np.sum(cnt * w_ * w_)
                + 0.5 * lam_v * np.sum(cnt[:, None] * V_ * V_)) / n

    hfd = 1e-6
    g_w0 = (fw_obj(w0 + hfd, w, V) - fw_obj(w0 - hfd, w, V)) / (2 * hfd)
    g_w = np.zeros(d)
    g_V = np.zeros((d, K))
    for j in range(d):
        e = np.zeros(d); e[j] = hfd
        g_w[j] = (fw_obj(w0, w + e, V) - fw_obj(w0, w - e, V)) / (2 * hfd)
        for k in range(K):
            E = np.zeros((d, K)); E[j, k] = hfd
            g_V[j, k] = (fw_obj(w0, w, V + E) - fw_obj(w0, w, V - E)) / (2 * hfd)

    errs = []
    for eta in (1e-2, 5e-3):
        o = O.Oracle(n, d, K, p, loss, lam_w, lam_v, eta, seed=3)
        o.w0, o.w[:], o.V[:] = w0, w, V
        o.load_csr(indptr, indices, vals, y)
        o.epoch()
        err = max(abs((o.w0 - w0) / eta + g_w0), np.abs((o.w - w) / eta + g_w).max(),
                  np.abs((o.V - V) / eta + g_V).max())
        errs.append(err)
    scale = max(abs(g_w0), np.abs(g_w).max(), np.abs(g_V).max())
    assert errs[0] < 0.05 * scale and errs[1] < 0.6 * errs[0] + 1e-7 * scale


@pytest.mark.parametrize("loss", [O.SQUARED, O.LOGISTIC])
def test_zero_factors_reduce_to_batch_gradient_descent_on_linear_model(loss):
    # V = 0 => a = 0 => every factor increment is 0; with lambda_w = 0 the epoch is exactly
    # w <- w - eta_s X^T G, w0 <- w0 - eta_s sum G  (least squares / logistic regression batch GD),
    # independent of p and of the visiting order.
    n, d, K = 23, 6, 3
    rng = np.random.default_rng(77)
    X, mask, indptr, indices, vals, w0, w, V = tiny_problem(rng, n, d, K, 0.5)
    y = (np.where(rng.random(n) < 0.5, 1.0, -1.0) if loss else rng.standard_normal(n)).astype(np.float32)
    yd = y.astype(np.float64)
    f = w0 + X @ w
    G = f - yd if loss == O.SQUARED else -yd / (1 + np.exp(yd * f))
    eta = 0.2
    want_w = w - eta / n * (X.T @ G)
    want_w0 = w0 - eta / n * G.sum()
    for p in (1, 2, 5):
        o = O.Oracle(n, d, K, p, loss, 0.0, 0.3, eta, seed=3)
        o.w0, o.w[:], o.V[:] = w0, w, 0.0
        o.load_csr(indptr, indices, vals, y)
        o.epoch()
        assert not o.V.any()
        np.testing.assert_allclose(o.w, want_w, rtol=1e-12, atol=1e-15)
        assert o.w0 == pytest.approx(want_w0, rel=1e-13)


def test_order_matters_for_factors_but_not_for_unregularised_weights():
    n, d, K = 37, 9, 3
    outs = {}
    for p in (1, 2, 4):
        o, *_ = _setup(5, n, d, K, p, O.LOGISTIC, lam=(0.0, 1e-2), eta=2.0)
        o.epoch()
        outs[p] = (o.w.copy(), o.V.copy())
    np.testing.assert_allclose(outs[1][0], outs[2][0], rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(outs[1][0], outs[4][0], rtol=1e-12, atol=1e-15)
    assert not np.allclose(outs[1][1], outs[4][1], rtol=1e-9, atol=0)


@pytest.mark.parametrize("loss,p", [(O.SQUARED, 4), (O.LOGISTIC, 3)])
def test_single_column_epoch_equals_full_epoch(loss, p):
    # columns do not interact while the auxiliaries are frozen, so the one-column routine used to
    # spot-check full-size runs must reproduce the full epoch's column exactly
    n, d, K = 45, 10, 4
    o, X, mask, y = _setup(11, n, d, K, p, loss)
    w0, w, V = o.w0, o.w.copy(), o.V.copy()
    o.epoch()
    for j in range(d):
        wj, vj, cnt = O.column_epoch(n, d, K, p, loss, o.eta_s, o.lambda_w, o.lambda_v, o.indptr, o.indices,
                                     o.values, o.y, w0, w, V, j)
        assert cnt == mask[:, j].sum()
        assert wj == pytest.approx(o.w[j], rel=1e-12, abs=1e-15)
        np.testing.assert_allclose(vj, o.V[j], rtol=1e-12, atol=1e-15)


def test_w0_step_uses_frozen_multipliers():
    o, *_ = _setup(3, 20, 6, 2, 2, O.SQUARED)
    w0, sg = o.w0, o.G.sum()
    o.epoch()
    assert o.w0 == pytest.approx(w0 - o.eta_s * sg, rel=1e-13)


def test_objective_decreases_on_small_workload():
    wl = W.make("C1")
    o = O.Oracle(wl.n, wl.d, wl.K, wl.p, wl.loss, wl.lambda_w, wl.lambda_v, wl.eta, wl.init_seed)
    o.load_csr(wl.indptr, wl.indices, wl.values, wl.y)
    objs = [o.objective] + [o.epoch() for _ in range(wl.epochs)]
    assert all(b < a for a, b in zip(objs, objs[1:]))
    assert np.isfinite(objs).all()


# ---- second schedule: auxiliaries recomputed after every R inner rounds ----

def test_segmented_epoch_with_one_segment_is_the_plain_epoch():
    for every in (0, 4, 9):
        a, *_ = _setup(11, 30, 8, 3, 4, O.LOGISTIC)
        b, *_ = _setup(11, 30, 8, 3, 4, O.LOGISTIC)
        for _ in range(2):
            a.epoch()
            b.epoch_segmented(every)
        assert a.w0 == b.w0 and np.array_equal(a.w, b.w) and np.array_equal(a.V, b.V)
        assert a.objective == b.objective


@pytest.mark.parametrize("loss,p,every", [(O.SQUARED, 4, 1), (O.LOGISTIC, 5, 2), (O.SQUARED, 3, 2)])
def test_segmented_epoch_on_linear_model_is_block_gradient_descent(loss, p, every):
    # V = 0 stays 0, and with lambda_w = 0 every segment is: G from the current (w0, w); then
    # w[column block c] -= eta_s X[row block r, column block c]^T G[row block r] for the tiles
    # (r, c = (r+s) mod p) of its rounds; w0 -= eta_s (rounds/p) sum G.  Written with dense numpy
    # blocks, independent of the oracle's tile lists.
    n, d, K = 26, 9, 2
    rng = np.random.default_rng(91 + p)
    X, mask, indptr, indices, vals, w0, w, V = tiny_problem(rng, n, d, K, 0.5)
    y = (np.where(rng.random(n) < 0.5, 1.0, -1.0) if loss else rng.standard_normal(n)).astype(np.float32)
    yd = y.astype(np.float64)
    eta = 0.3
    o = O.Oracle(n, d, K, p, loss, 0.0, 0.2, eta, seed=3)
    o.w0, o.w[:], o.V[:] = w0, w, 0.0
    o.load_csr(indptr, indices, vals, y)
    o.epoch_segmented(every)
    rb = np.arange(n) * p // n
    cb = np.arange(d) * p // d
    ww, ww0 = w.copy(), w0
    for s0 in range(0, p, every):
        s1 = min(s0 + every, p)
        f = ww0 + X @ ww
        G = f - yd if loss == O.SQUARED else -yd / (1 + np.exp(yd * f))
        ww0 -= eta / n * (s1 - s0) / p * G.sum()
        for s in range(s0, s1):
            for r in range(p):
                c = (r + s) % p
                rows, cols = np.nonzero(rb == r)[0], np.nonzero(cb == c)[0]
                ww[cols] -= eta / n * (X[np.ix_(rows, cols)].T @ G[rows])
    assert not o.V.any()
    np.testing.assert_allclose(o.w, ww, rtol=1e-12, atol=1e-15)
    assert o.w0 == pytest.approx(ww0, rel=1e-13)
    # and it is not the plain epoch: the later segments saw fresher multipliers
    o2 = O.Oracle(n, d, K, p, loss, 0.0, 0.2, eta, seed=3)
    o2.w0, o2.w[:], o2.V[:] = w0, w, 0.0
    o2.load_csr(indptr, indices, vals, y)
    o2.epoch()
    assert np.abs(o2.w - o.w).max() > 1e-6


def test_segmented_epoch_recomputes_auxiliaries_between_segments():
    # after a segmented epoch the stored auxiliaries are consistent with the final parameters, and the
    # factor rows differ from the plain epoch's (the second segment used a_i of the updated V)
    a, X, mask, *_ = _setup(13, 40, 9, 3, 4, O.SQUARED)
    b, *_ = _setup(13, 40, 9, 3, 4, O.SQUARED)
    a.epoch()
    b.epoch_segmented(2)
    np.testing.assert_allclose(b.A, X @ b.V, rtol=1e-12, atol=1e-14)
    assert np.abs(a.V - b.V).max() > 1e-9


def test_segmented_schedule_converges_at_least_as_fast_on_small_workload():
    wl = W.make("C1")
    objs = {}
    for every in (0, 1):
        o = O.Oracle(wl.n, wl.d, wl.K, wl.p, wl.loss, wl.lambda_w, wl.lambda_v, 2.0, wl.init_seed)
        o.load_csr(wl.indptr, wl.indices, wl.values, wl.y)
        for _ in range(10):
            o.epoch_segmented(every)
        objs[every] = o.objective
    assert np.isfinite(objs[1]) and objs[1] <= objs[0] * 1.001
