"""Failure path of the stratum SGD launch, exercised without faulting or hanging anything, and the
bounds-checked build of the library.

A chunk that waits for more finished chunks than its column block will ever report cannot go on: its wait
is bounded, so it gives up after a few polls, every warp leaves at its next ticket, and the host is told."""
import numpy as np
import pytest

from oracle import dsfacto_oracle as O
from paper_2004_13940_b200 import dsfacto as D
from paper_2004_13940_b200 import workloads as W

pytestmark = pytest.mark.gpu


def test_a_wait_that_cannot_end_gives_up_and_the_handle_recovers():
    wl = W.make("C1")
    g = D.DSFacto(wl.n, wl.d, wl.K, wl.p, wl.loss, wl.lambda_w, wl.lambda_v, wl.eta, wl.init_seed)
    g.debug_set(D.DEBUG_SPIN_LIMIT, 32)            # a few polls of about 200 ns each
    g.debug_set(D.DEBUG_EXTRA_NEED, 1 << 20)       # more chunks than the data set has
    g.load_csr(wl.indptr, wl.indices, wl.values, wl.y)
    w0, w, V = g.get_params()
    obj0 = g.objective()
    assert D.dsfacto_epoch(g._h) == D.ERR_CUDA
    assert b"timed out" in D.lib().dsfacto_last_error(g._h)
    # the handle refuses further epochs until its parameters are replaced
    assert D.dsfacto_epoch(g._h) == D.ERR_CUDA
    assert b"gave up" in D.lib().dsfacto_last_error(g._h)
    # recovery: no planted wait at the next load, parameters restored, data loaded again
    g.debug_set(D.DEBUG_EXTRA_NEED, 0)
    g.debug_set(D.DEBUG_SPIN_LIMIT, 1 << 22)
    g.set_params(w0, w, V)
    g.load_csr(wl.indptr, wl.indices, wl.values, wl.y)
    assert g.objective() == pytest.approx(obj0, rel=1e-12)
    o = O.Oracle(wl.n, wl.d, wl.K, wl.p, wl.loss, wl.lambda_w, wl.lambda_v, wl.eta, wl.init_seed)
    o.load_csr(wl.indptr, wl.indices, wl.values, wl.y)
    for _ in range(3):
        assert g.epoch() == pytest.approx(o.epoch(), rel=1e-4)
    w0b, wb, Vb = g.get_params()
    assert np.abs(wb - o.w).max() <= 1e-4 * (1 + np.abs(o.w).max())
    assert np.all(np.abs(Vb - o.V) <= 1e-4 * (1 + np.abs(o.V)))
    g.close()
    # and a fresh handle is not affected by what happened to the other one
    with D.DSFacto(wl.n, wl.d, wl.K, wl.p, wl.loss, wl.lambda_w, wl.lambda_v, wl.eta, wl.init_seed) as h:
        h.load_csr(wl.indptr, wl.indices, wl.values, wl.y)
        o2 = O.Oracle(wl.n, wl.d, wl.K, wl.p, wl.loss, wl.lambda_w, wl.lambda_v, wl.eta, wl.init_seed)
        o2.load_csr(wl.indptr, wl.indices, wl.values, wl.y)
        assert h.epoch() == pytest.approx(o2.epoch(), rel=1e-4)


def test_debug_knobs_reject_bad_values():
    wl = W.make("C1")
    with D.DSFacto(wl.n, wl.d, wl.K, wl.p, wl.loss, wl.lambda_w, wl.lambda_v, wl.eta, wl.init_seed) as g:
        assert D.dsfacto_debug_set(g._h, D.DEBUG_SPIN_LIMIT, 0) == D.ERR_INVALID_ARG
        assert D.dsfacto_debug_set(g._h, D.DEBUG_CHUNK_LEN, 7) == D.ERR_INVALID_ARG
        assert D.dsfacto_debug_set(g._h, D.DEBUG_CHUNK_LEN, 4097) == D.ERR_INVALID_ARG
        assert D.dsfacto_debug_set(g._h, 99, 1) == D.ERR_INVALID_ARG
        assert D.dsfacto_debug_set(g._h, D.DEBUG_CHUNK_LEN, 64) == D.OK
        g.load_csr(wl.indptr, wl.indices, wl.values, wl.y)
        o = O.Oracle(wl.n, wl.d, wl.K, wl.p, wl.loss, wl.lambda_w, wl.lambda_v, wl.eta, wl.init_seed)
        o.load_csr(wl.indptr, wl.indices, wl.values, wl.y)
        assert g.epoch() == pytest.approx(o.epoch(), rel=1e-4)


@pytest.mark.parametrize("name,epochs", [("C1", 3), ("C2", 2), ("C3", 2), ("C5s", 1)])
def test_bounds_checked_build_finds_nothing_and_matches_the_oracle(name, epochs):
    # libdsfacto_debug.so checks every row, column, chunk and run index the stratum SGD kernel forms; a bad
    # index would make dsfacto_epoch return DSFACTO_ERR_CUDA with the failed check in the error text
    wl = W.make(name)
    o = O.Oracle(wl.n, wl.d, wl.K, wl.p, wl.loss, wl.lambda_w, wl.lambda_v, wl.eta, wl.init_seed)
    o.load_csr(wl.indptr, wl.indices, wl.values, wl.y)
    with D.use_debug_library():
        with D.DSFacto(wl.n, wl.d, wl.K, wl.p, wl.loss, wl.lambda_w, wl.lambda_v, wl.eta, wl.init_seed) as g:
            g.load_csr(wl.indptr, wl.indices, wl.values, wl.y)
            for _ in range(epochs):
                assert g.epoch() == pytest.approx(o.epoch(), rel=1e-4)
            w0, w, V = g.get_params()
    assert np.abs(w - o.w).max() <= 1e-4 * (1 + np.abs(o.w).max())
    assert np.all(np.abs(V - o.V) <= 1e-4 * (1 + np.abs(o.V)))
