"""Pins for the oracle's model side: score, auxiliaries, multiplier, objective, initialisation.

Each test compares the oracle with something that is not the oracle: the pairwise definition by
brute force, hand-worked numbers, finite differences, or the published SplitMix64 vectors."""
import math

import numpy as np
import pytest

from oracle import dsfacto_oracle as O
from tests.helpers import fm_pairwise, loss_np, objective_np, read_golden, tiny_problem


def _oracle_on(n, d, K, p, loss, indptr, indices, vals, y, w0, w, V, lam=(1e-3, 1e-3), eta=0.01):
    o = O.Oracle(n, d, K, p, loss, lam[0], lam[1], eta, seed=1)
    o.w0, o.w[:], o.V[:] = w0, w, V
    o.load_csr(indptr, indices, vals, y)
    return o


@pytest.mark.parametrize("seed,n,d,K,density", [(0, 7, 5, 3, 0.6), (1, 12, 9, 4, 0.4), (2, 5, 6, 1, 1.0),
                                                (3, 9, 4, 7, 0.5)])
def test_score_equals_pairwise_definition(seed, n, d, K, density):
    # eq. (fm_model2) must reproduce eq. (fm_model) (the O(K nnz^2) pairwise sum)
    rng = np.random.default_rng(seed)
    X, mask, indptr, indices, vals, w0, w, V = tiny_problem(rng, n, d, K, density)
    got = O.score(indptr, indices, vals, w0, w, V)
    want = fm_pairwise(X, mask, w0, w, V)
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-12)


def test_hand_worked_example():
    rows = read_golden("fm_hand_example.txt")
    w0 = 0.5
    w = np.array([1.0, -2.0, 0.25])
    V = np.array([[1.0, 0.0], [0.5, 1.0], [-1.0, 2.0]])
    X = np.array([[1, 2, 0], [0, 1, -1], [2, 1, 3]], np.float64)
    y = np.array([1, -1, 1], np.float32)
    indptr = np.array([0, 2, 4, 7], np.int64)
    indices = np.array([0, 1, 1, 2, 0, 1, 2], np.int32)
    vals = np.array([1, 2, 1, -1, 2, 1, 3], np.float32)
    o = _oracle_on(3, 3, 2, 1, O.SQUARED, indptr, indices, vals, y, w0, w, V)
    for i, (_, f, a1, a2, g) in enumerate(rows):
        assert o.f[i] == pytest.approx(float(f), abs=1e-14)
        assert o.A[i, 0] == pytest.approx(float(a1), abs=1e-14)
        assert o.A[i, 1] == pytest.approx(float(a2), abs=1e-14)
        assert o.G[i] == pytest.approx(float(g), abs=1e-14)
    o2 = _oracle_on(3, 3, 2, 1, O.LOGISTIC, indptr, indices, vals, y, w0, w, V)
    want = [-1 / (1 + math.exp(-1.5)), 1 / (1 + math.exp(3.25)), -1 / (1 + math.exp(0.75))]
    np.testing.assert_allclose(o2.G, want, rtol=1e-14)


@pytest.mark.parametrize("loss", [O.SQUARED, O.LOGISTIC])
def test_objective_and_reformulation_invariant(loss):
    # objective eq. (fm_obj) from the oracle == brute force from (w, V); and the doubly-separable
    # form written with the stored auxiliaries (lin, A, q) gives the same value only while the
    # auxiliaries are consistent with V
    rng = np.random.default_rng(10 + loss)
    n, d, K = 11, 6, 3
    X, mask, indptr, indices, vals, w0, w, V = tiny_problem(rng, n, d, K, 0.5)
    y = np.where(rng.random(n) < 0.5, 1.0, -1.0).astype(np.float32) if loss else rng.standard_normal(n).astype(np.float32)
    lam_w, lam_v = 0.03, 0.07
    o = _oracle_on(n, d, K, 2, loss, indptr, indices, vals, y, w0, w, V, lam=(lam_w, lam_v))
    want = objective_np(X, mask, y.astype(np.float64), loss, w0, w, V, lam_w, lam_v)
    assert o.objective == pytest.approx(want, rel=1e-12)

    def separable(A):
        f = o.w0 + o.lin + 0.5 * ((A * A).sum(1) - o.q)
        return loss_np(loss, f, y.astype(np.float64)).mean() + 0.5 * lam_w * np.sum(w * w) + 0.5 * lam_v * np.sum(V * V)

    assert separable(o.A) == pytest.approx(want, rel=1e-12)
    np.testing.assert_allclose(o.A, X @ V, rtol=1e-12, atol=1e-14)          # eq. (compute_a_jk)
    np.testing.assert_allclose(o.lin, X @ w, rtol=1e-12, atol=1e-14)
    assert abs(separable(o.A + 0.05) - want) > 1e-4                          # negative control
    assert o.mean_loss == pytest.approx(loss_np(loss, fm_pairwise(X, mask, w0, w, V), y.astype(np.float64)).mean(), rel=1e-12)


@pytest.mark.parametrize("loss", [O.SQUARED, O.LOGISTIC])
def test_multiplier_is_loss_derivative(loss):
    # G_i = dl_i/df_i; since df/dw0 = 1, a central difference of the per-row loss in w0 gives G_i
    rng = np.random.default_rng(20 + loss)
    n, d, K = 9, 5, 2
    X, mask, indptr, indices, vals, w0, w, V = tiny_problem(rng, n, d, K, 0.6)
    y = np.where(rng.random(n) < 0.5, 1.0, -1.0).astype(np.float32) if loss else rng.standard_normal(n).astype(np.float32)
    o = _oracle_on(n, d, K, 1, loss, indptr, indices, vals, y, w0, w, V)
    h = 1e-6
    lp = loss_np(loss, fm_pairwise(X, mask, w0 + h, w, V), y.astype(np.float64))
    lm = loss_np(loss, fm_pairwise(X, mask, w0 - h, w, V), y.astype(np.float64))
    np.testing.assert_allclose(o.G, (lp - lm) / (2 * h), rtol=1e-6, atol=1e-8)
    assert o.sum_G == pytest.approx(o.G.sum(), rel=1e-13)


def test_logistic_loss_is_stable_for_large_margins():
    indptr = np.array([0, 1, 2], np.int64)
    indices = np.array([0, 0], np.int32)
    vals = np.array([1.0, 1.0], np.float32)
    y = np.array([1.0, -1.0], np.float32)
    o = _oracle_on(2, 1, 1, 1, O.LOGISTIC, indptr, indices, vals, y, 0.0, np.array([800.0]), np.zeros((1, 1)))
    assert np.isfinite(o.lossv).all() and np.isfinite(o.G).all()
    assert o.lossv[0] == pytest.approx(0.0, abs=1e-300) and o.lossv[1] == pytest.approx(800.0)
    assert o.G[0] == pytest.approx(0.0, abs=1e-300) and o.G[1] == pytest.approx(1.0)


def test_splitmix64_published_vectors():
    for seed, c, value in read_golden("splitmix64_vectors.txt"):
        assert O.lib().oracle_splitmix64_at(int(seed), int(c)) == int(value)


def test_init_is_seeded_normal_with_sigma_001():
    w0, w, V = O.init_params(4000, 8, seed=2004)
    assert w0 == 0.0 and not w.any()
    assert abs(V.mean()) < 3 * 0.01 / math.sqrt(V.size)
    assert V.std() == pytest.approx(0.01, rel=0.02)
    assert np.array_equal(V, V.astype(np.float32).astype(np.float64))      # fp32-representable
    # element e = j*K+k is Box-Muller (cosine branch) of stream outputs 2e, 2e+1
    e = 5 * 8 + 3
    u1 = ((O.lib().oracle_splitmix64_at(2004, 2 * e) >> 11) + 0.5) / 2.0 ** 53
    u2 = ((O.lib().oracle_splitmix64_at(2004, 2 * e + 1) >> 11) + 0.5) / 2.0 ** 53
    z = math.sqrt(-2 * math.log(u1)) * math.cos(2 * math.pi * u2)
    assert V[5, 3] == pytest.approx(float(np.float32(0.01 * z)), rel=1e-6)
    # 4-sigma tail fraction of a normal: 6.3e-5; a uniform or wrong-variance draw would miss this
    assert (np.abs(V) > 0.04).mean() < 5e-4 and (np.abs(V) > 0.02).mean() == pytest.approx(0.0455, rel=0.1)
    assert not np.array_equal(V, O.init_params(4000, 8, seed=2005)[2])


@pytest.mark.parametrize("loss", [O.SQUARED, O.LOGISTIC])
def test_heldout_evaluation_matches_library_metrics(loss):
    # mean loss, RMSE and accuracy of held-out rows against scikit-learn's metric routines applied
    # to brute-force pairwise scores (eq. (fm_model)); a flipped label must change the answer
    from sklearn.metrics import accuracy_score, log_loss, mean_squared_error

    rng = np.random.default_rng(40 + loss)
    n, d, K = 23, 7, 3
    X, mask, indptr, indices, vals, w0, w, V = tiny_problem(rng, n, d, K, 0.6)
    f = fm_pairwise(X, mask, w0, w, V)
    if loss == O.SQUARED:
        y = (f + rng.standard_normal(n)).astype(np.float32)
        mean_loss, rmse = O.evaluate(loss, indptr, indices, vals, y, w0, w, V)
        mse = mean_squared_error(y.astype(np.float64), f)
        assert rmse == pytest.approx(math.sqrt(mse), rel=1e-12)
        assert mean_loss == pytest.approx(0.5 * mse, rel=1e-12)
        y2 = y.copy(); y2[3] += 1.0
        assert O.evaluate(loss, indptr, indices, vals, y2, w0, w, V)[1] != pytest.approx(rmse, rel=1e-6)
    else:
        y = np.where(rng.random(n) < 0.5, 1.0, -1.0).astype(np.float32)
        mean_loss, acc = O.evaluate(loss, indptr, indices, vals, y, w0, w, V)
        assert acc == pytest.approx(accuracy_score(y, np.where(f > 0, 1.0, -1.0)), abs=1e-15)
        prob = 1.0 / (1.0 + np.exp(-f))                                    # P(y = +1 | x) under the logistic model
        assert mean_loss == pytest.approx(log_loss(y, prob, labels=[-1.0, 1.0]), rel=1e-10)
        y2 = y.copy(); y2[3] = -y2[3]
        assert abs(O.evaluate(loss, indptr, indices, vals, y2, w0, w, V)[1] - acc) == pytest.approx(1.0 / n, rel=1e-9)


def test_heldout_accuracy_counts_zero_score_as_wrong():
    # w = 0, V = 0, w0 = 0: every score is exactly 0, which predicts neither class
    indptr = np.array([0, 1, 2], np.int64)
    indices = np.array([0, 1], np.int32)
    vals = np.array([1.0, 2.0], np.float32)
    y = np.array([1.0, -1.0], np.float32)
    mean_loss, acc = O.evaluate(O.LOGISTIC, indptr, indices, vals, y, 0.0, np.zeros(2), np.zeros((2, 2)))
    assert acc == 0.0 and mean_loss == pytest.approx(math.log(2.0), rel=1e-15)
