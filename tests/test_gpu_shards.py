"""Column shards (Section 4.2's column blocks spread over workers) emulated on one GPU: several shard handles
in one process, their partial auxiliaries [A | lin | q] added on the device, against the oracle's plain epoch.

Tolerances are those of tests/test_gpu_parity.py; the shards add their partial sums in fp32, which reorders
sums that the single handle forms in one go, well inside 2e-5 (1 + |ref|)."""
import numpy as np
import pytest

from oracle import dsfacto_oracle as O
from paper_2004_13940_b200 import dsfacto as D
from paper_2004_13940_b200 import sharded as S
from paper_2004_13940_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,nshards,epochs", [("C1", 2, 4), ("C1", 3, 2), ("C2", 2, 3), ("C3", 2, 3), ("C3", 5, 2),
                                                 ("C4s", 2, 2), ("C5s", 4, 1)])
def test_sharded_epochs_match_the_oracle(name, nshards, epochs):
    wl = W.make(name)
    o = O.Oracle(wl.n, wl.d, wl.K, wl.p, wl.loss, wl.lambda_w, wl.lambda_v, wl.eta, wl.init_seed)
    o.load_csr(wl.indptr, wl.indices, wl.values, wl.y)
    with S.ShardGroup(wl.n, wl.d, wl.K, wl.p, wl.loss, wl.lambda_w, wl.lambda_v, wl.eta, wl.init_seed, nshards) as g:
        assert g.load_csr(wl.indptr, wl.indices, wl.values, wl.y) == pytest.approx(o.objective, rel=1e-5)
        # the shards' column ranges partition the columns, and their tile lists are the oracle's restricted to them
        ranges = [s.h.shard_columns() for s in g.shards]
        assert ranges[0][0] == 0 and ranges[-1][1] == wl.d and all(a[1] == b[0] for a, b in zip(ranges, ranges[1:]))
        for s, (lo, hi) in zip(g.shards, ranges):
            tp, rows, cols, vals = s.h.get_tiles()
            keep = (o.cols >= lo) & (o.cols < hi)
            assert np.array_equal(rows, o.rows[keep]) and np.array_equal(cols, o.cols[keep])
            assert np.array_equal(vals.view(np.uint32), o.vals[keep].view(np.uint32))
        A, G = g.get_aux()
        np.testing.assert_allclose(A, o.A, rtol=0, atol=2e-5 * (1 + np.abs(o.A).max()))
        np.testing.assert_allclose(G, o.G, rtol=0, atol=2e-5 * (1 + np.abs(o.G).max()))
        for e in range(epochs):
            before = (o.w.copy(), o.V.copy())
            want, got = o.epoch(), g.epoch()
            assert got == pytest.approx(want, rel=1e-4), e
            w0, w, V = g.get_params()
            assert abs(w0 - o.w0) <= 1e-4 * (1 + abs(o.w0))
            assert np.abs(w - o.w).max() <= 1e-4 * (1 + np.abs(o.w).max())
            assert np.all(np.abs(V - o.V) <= 1e-4 * (1 + np.abs(o.V)))
            if e == 0:
                for got_p, ref, start in ((w, o.w, before[0]), (V, o.V, before[1])):
                    dref = ref - start
                    assert np.abs(got_p.astype(np.float64) - start - dref).max() <= 2e-3 * np.abs(dref).max() + 2e-7
        A, G = g.get_aux()
        np.testing.assert_allclose(A, o.A, rtol=0, atol=2e-5 * (1 + np.abs(o.A).max()))
        np.testing.assert_allclose(G, o.G, rtol=0, atol=2e-5 * (1 + np.abs(o.G).max()))


def test_shard_calls_are_refused_where_they_do_not_apply():
    wl = W.make("C1")
    with D.DSFacto(wl.n, wl.d, wl.K, wl.p, wl.loss, wl.lambda_w, wl.lambda_v, wl.eta, wl.init_seed) as g:
        g.load_csr(wl.indptr, wl.indices, wl.values, wl.y)
        assert D.lib().dsfacto_shard_epoch_begin(g._h) == D.ERR_INVALID_ARG         # not a shard
    with D.DSFacto(wl.n, wl.d, wl.K, wl.p, wl.loss, wl.lambda_w, wl.lambda_v, wl.eta, wl.init_seed, shard=1, nshards=2) as s:
        assert D.dsfacto_set_refresh_every(s._h, 2) == D.ERR_INVALID_ARG
        s.load_csr(wl.indptr, wl.indices, wl.values, wl.y)
        assert D.dsfacto_epoch(s._h) == D.ERR_INVALID_ARG                             # a shard cannot finish an epoch alone
        assert D.lib().dsfacto_shard_epoch_begin(s._h) == D.ERR_INVALID_ARG         # the first sums are still owed
    bad = D._vp()
    assert D.lib().dsfacto_create_shard(D.ctypes.byref(bad), 100, 10, 4, 2, 0, 0.0, 0.0, 0.1, 1, 0, 3) == D.ERR_INVALID_ARG
    assert D.lib().dsfacto_create_shard(D.ctypes.byref(bad), 100, 10, 4, 2, 0, 0.0, 0.0, 0.1, 1, 2, 2) == D.ERR_INVALID_ARG
