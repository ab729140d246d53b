"""Held-out evaluation and learning-rate changes of the CUDA path against the CPU oracle.

Rows [0, n) of a workload train, rows [n, n+m) of the same generator (same planted model) are the
held-out set.  Tolerances: mean loss and RMSE are fp64 sums of fp32 per-row terms -> 1e-5 relative;
the accuracy is a count decided by the sign of an fp32 score, so the two sides may differ on rows
whose reference score lies within the score tolerance 2e-5 (1 + max|f|) of zero, and on no others."""
import numpy as np
import pytest

from oracle import dsfacto_oracle as O
from paper_2004_13940_b200 import dsfacto as D
from paper_2004_13940_b200 import workloads as W

pytestmark = pytest.mark.gpu


def split(name, n, m):
    wl = W.make(name, n=n + m)
    cut = int(wl.indptr[n])
    train = (wl.indptr[: n + 1].copy(), wl.indices[:cut], wl.values[:cut], wl.y[:n])
    held = ((wl.indptr[n:] - cut).astype(np.int64), wl.indices[cut:], wl.values[cut:], wl.y[n:])
    return wl, train, held


@pytest.mark.parametrize("name,n,m,epochs", [("C1", 2000, 500, 3), ("C2", 50_000, 10_000, 3), ("C3", 20_000, 5_000, 2),
                                             ("C4s", 100_000, 30_000, 1), ("C5s", 20_000, 3_000, 1)])
def test_heldout_metrics_match_oracle(name, n, m, epochs):
    wl, train, held = split(name, n, m)
    o = O.Oracle(n, wl.d, wl.K, wl.p, wl.loss, wl.lambda_w, wl.lambda_v, wl.eta, wl.init_seed)
    o.load_csr(*train)
    with D.DSFacto(n, wl.d, wl.K, wl.p, wl.loss, wl.lambda_w, wl.lambda_v, wl.eta, wl.init_seed) as g:
        g.load_csr(*train)
        for e in range(epochs + 1):
            ref_loss, ref_metric = o.evaluate(*held)
            got_loss, got_metric = g.evaluate(*held)
            assert got_loss == pytest.approx(ref_loss, rel=1e-5, abs=1e-7)
            if wl.loss == W.SQUARED:
                assert got_metric == pytest.approx(ref_metric, rel=1e-5)
            else:
                f = o.predict(*held[:3])
                near_zero = int(np.count_nonzero(np.abs(f) <= 2e-5 * (1 + np.abs(f).max())))
                assert abs(got_metric - ref_metric) * m <= near_zero + 1e-9
            if e < epochs:
                want, got = o.epoch(), g.epoch()
                assert got == pytest.approx(want, rel=1e-4)
        # evaluating leaves the training state alone
        obj = g.objective()
        g.evaluate(*held)
        assert g.objective() == obj
        A, G = g.get_aux()
        np.testing.assert_allclose(A, o.A, rtol=0, atol=2e-5 * (1 + np.abs(o.A).max()))


def test_evaluate_on_training_rows_reproduces_the_training_loss():
    wl = W.make("C2")
    with D.DSFacto(wl.n, wl.d, wl.K, wl.p, wl.loss, wl.lambda_w, wl.lambda_v, wl.eta, wl.init_seed) as g:
        g.load_csr(wl.indptr, wl.indices, wl.values, wl.y)
        g.epoch()
        mean_loss, acc = g.evaluate(wl.indptr, wl.indices, wl.values, wl.y)
        assert mean_loss == pytest.approx(g.stats()[0], rel=1e-12)
        f = g.predict()
        assert acc == pytest.approx(np.mean(wl.y * f > 0), abs=1e-12)


def test_learning_rate_schedule_matches_oracle():
    wl = W.make("C1")
    o = O.Oracle(wl.n, wl.d, wl.K, wl.p, wl.loss, wl.lambda_w, wl.lambda_v, 2.0, wl.init_seed)
    o.load_csr(wl.indptr, wl.indices, wl.values, wl.y)
    with D.DSFacto(wl.n, wl.d, wl.K, wl.p, wl.loss, wl.lambda_w, wl.lambda_v, 2.0, wl.init_seed) as g:
        g.load_csr(wl.indptr, wl.indices, wl.values, wl.y)
        for t in range(6):
            eta = 2.0 / (1.0 + 0.5 * t)
            o.set_eta(eta)
            g.set_eta(eta)
            want, got = o.epoch(), g.epoch()
            assert got == pytest.approx(want, rel=1e-4)
        w0, w, V = g.get_params()
        assert np.abs(w - o.w).max() <= 1e-4 * (1 + np.abs(o.w).max())
        assert np.all(np.abs(V - o.V) <= 1e-4 * (1 + np.abs(o.V)))
        # a different schedule gives a different trajectory (the setter is not ignored)
    o2 = O.Oracle(wl.n, wl.d, wl.K, wl.p, wl.loss, wl.lambda_w, wl.lambda_v, 2.0, wl.init_seed)
    o2.load_csr(wl.indptr, wl.indices, wl.values, wl.y)
    for t in range(6):
        o2.epoch()
    assert abs(o2.objective - o.objective) > 1e-3 * abs(o.objective)


def test_evaluate_argument_checks():
    wl = W.make("C1")
    with D.DSFacto(wl.n, wl.d, wl.K, wl.p, wl.loss, wl.lambda_w, wl.lambda_v, wl.eta, wl.init_seed) as g:
        rc, _, _ = D.dsfacto_evaluate(g._h, wl.n, None, None, None, wl.y)
        assert rc == D.ERR_INVALID_ARG
        rc, _, _ = D.dsfacto_evaluate(g._h, 0, wl.indptr, wl.indices, wl.values, wl.y)
        assert rc == D.ERR_INVALID_ARG
        bad_y = wl.y.copy(); bad_y[5] = np.nan
        rc, _, _ = D.dsfacto_evaluate(g._h, wl.n, wl.indptr, wl.indices, wl.values, bad_y)
        assert rc == D.ERR_INVALID_CSR
        bad_idx = wl.indices.copy(); bad_idx[0] = wl.d
        rc, _, _ = D.dsfacto_evaluate(g._h, wl.n, wl.indptr, bad_idx, wl.values, wl.y)
        assert rc == D.ERR_INVALID_CSR
        # works before any training data is loaded: it needs parameters only
        rc, ml, mt = D.dsfacto_evaluate(g._h, wl.n, wl.indptr, wl.indices, wl.values, wl.y)
        assert rc == D.OK and np.isfinite(ml) and np.isfinite(mt)
        assert D.dsfacto_set_eta(g._h, 0.0) == D.ERR_INVALID_ARG
        assert D.dsfacto_set_eta(g._h, float("nan")) == D.ERR_INVALID_ARG
