"""Column slots of the recompute pass: the device copy of the CSR may number the columns by frequency and
read w and V from a copy in that order.  No sum changes its order, so every result must be bit-identical to
the same library with the renumbering switched off, and it must match the oracle as before."""
import numpy as np
import pytest

from oracle import dsfacto_oracle as O
from paper_2004_13940_b200 import dsfacto as D
from paper_2004_13940_b200 import workloads as W
from paper_2004_13940_b200.sharded import ShardGroup

pytestmark = pytest.mark.gpu

ON, OFF = 1, 2


def _run(wl, order, epochs, refresh_every=0):
    with D.DSFacto(wl.n, wl.d, wl.K, wl.p, wl.loss, wl.lambda_w, wl.lambda_v, wl.eta, wl.init_seed) as g:
        g.debug_set(D.DEBUG_COLUMN_ORDER, order)
        if refresh_every:
            g.set_refresh_every(refresh_every)
        g.load_csr(wl.indptr, wl.indices, wl.values, wl.y)
        objs = [g.objective()] + [g.epoch() for _ in range(epochs)]
        A, G = g.get_aux()
        w0, w, V = g.get_params()
        f = g.predict()
        launches = g.launch_count()
    return objs, A, G, w0, w, V, f, launches


@pytest.mark.parametrize("name,epochs", [("C1", 3), ("C2", 2), ("C3", 2), ("C4s", 1), ("C5s", 1)])
def test_renumbered_columns_change_no_bit(name, epochs):
    wl = W.make(name)
    on = _run(wl, ON, epochs)
    off = _run(wl, OFF, epochs)
    assert on[0] == off[0]
    for a, b in zip(on[1:7], off[1:7]):
        assert np.array_equal(np.asarray(a), np.asarray(b))
    # the renumbered handle really took the other way: two more kernels at the load, one more per pass
    assert on[7] > off[7]


@pytest.mark.parametrize("name", ["C2", "C3"])
def test_renumbered_columns_match_the_oracle(name):
    wl = W.make(name)
    o = O.Oracle(wl.n, wl.d, wl.K, wl.p, wl.loss, wl.lambda_w, wl.lambda_v, wl.eta, wl.init_seed)
    o.load_csr(wl.indptr, wl.indices, wl.values, wl.y)
    objs, A, G, w0, w, V, f, _ = _run(wl, ON, 2)
    assert objs[0] == pytest.approx(o.objective, rel=1e-5)
    for t in range(2):
        assert objs[t + 1] == pytest.approx(o.epoch(), rel=1e-4)
    assert np.abs(w - o.w).max() <= 1e-4 * (1 + np.abs(o.w).max())
    assert np.all(np.abs(V - o.V) <= 1e-4 * (1 + np.abs(o.V)))
    assert np.all(np.abs(G - o.G) <= 1e-4 * (1 + np.abs(o.G)))
    # held-out rows given by the caller keep the caller's column indices
    m = min(wl.n, 500)
    ip = wl.indptr[: m + 1]
    with D.DSFacto(wl.n, wl.d, wl.K, wl.p, wl.loss, wl.lambda_w, wl.lambda_v, wl.eta, wl.init_seed) as g:
        g.debug_set(D.DEBUG_COLUMN_ORDER, ON)
        g.load_csr(wl.indptr, wl.indices, wl.values, wl.y)
        g.epoch()
        all_rows = g.predict()
        some = g.predict(ip, wl.indices[: ip[-1]], wl.values[: ip[-1]])
    assert np.array_equal(all_rows[:m], some)


def test_renumbered_columns_with_the_second_schedule_and_with_shards():
    wl = W.make("C2")
    on = _run(wl, ON, 2, refresh_every=4)
    off = _run(wl, OFF, 2, refresh_every=4)
    assert on[0] == off[0]
    assert np.array_equal(on[5], off[5])
    res = []
    for order in (ON, OFF):
        grp = ShardGroup(wl.n, wl.d, wl.K, wl.p, wl.loss, wl.lambda_w, wl.lambda_v, wl.eta, wl.init_seed, nshards=3)
        for sh in grp.shards:
            sh.h.debug_set(D.DEBUG_COLUMN_ORDER, order)
        objs = [grp.load_csr(wl.indptr, wl.indices, wl.values, wl.y)] + [grp.epoch() for _ in range(2)]
        w0, w, V = grp.get_params()
        grp.close()
        res.append((objs, w, V))
    assert res[0][0] == res[1][0]
    assert np.array_equal(res[0][1], res[1][1]) and np.array_equal(res[0][2], res[1][2])


def test_knob_rejects_bad_values():
    wl = W.make("C1")
    with D.DSFacto(wl.n, wl.d, wl.K, wl.p, wl.loss, wl.lambda_w, wl.lambda_v, wl.eta, wl.init_seed) as g:
        assert D.dsfacto_debug_set(g._h, D.DEBUG_COLUMN_ORDER, 3) == D.ERR_INVALID_ARG
        assert D.dsfacto_debug_set(g._h, D.DEBUG_COLUMN_ORDER, -1) == D.ERR_INVALID_ARG
        assert D.dsfacto_debug_set(g._h, D.DEBUG_COLUMN_ORDER, 0) == D.OK
