"""Parity of the CUDA path (through the C ABI) against the CPU oracle, element by element, on the
same seeded inputs.

Tolerances (from the arithmetic; see the design notes):
  bucketing            bit-exact
  A, G, scores         fp32 sums of <= a few hundred products: 2e-5 * (1 + |ref|) absolute
  objective            1e-4 relative at every epoch (contract); observed ~1e-6
  parameters, 1 epoch  1e-4 * (1 + |ref|) max-abs (contract) AND, because one epoch moves the
                       parameters by little, the stricter |delta_gpu - delta_ref| <=
                       2e-3 * max|delta_ref| + 2e-7 on the per-epoch change
"""
import numpy as np
import pytest

from oracle import dsfacto_oracle as O
from paper_2004_13940_b200 import dsfacto as D
from paper_2004_13940_b200 import workloads as W

pytestmark = pytest.mark.gpu


def make_pair(wl, eta=None, K=None, p=None, lam=None):
    K = wl.K if K is None else K
    p = wl.p if p is None else p
    eta = wl.eta if eta is None else eta
    lw, lv = (wl.lambda_w, wl.lambda_v) if lam is None else lam
    o = O.Oracle(wl.n, wl.d, K, p, wl.loss, lw, lv, eta, wl.init_seed)
    o.load_csr(wl.indptr, wl.indices, wl.values, wl.y)
    g = D.DSFacto(wl.n, wl.d, K, p, wl.loss, lw, lv, eta, wl.init_seed)
    g.load_csr(wl.indptr, wl.indices, wl.values, wl.y)
    return o, g


def check_aux(o, g):
    A, G = g.get_aux()
    np.testing.assert_allclose(A, o.A, rtol=0, atol=2e-5 * (1 + np.abs(o.A).max()))
    np.testing.assert_allclose(G, o.G, rtol=0, atol=2e-5 * (1 + np.abs(o.G).max()))
    ml, sg = g.stats()
    assert ml == pytest.approx(o.mean_loss, rel=1e-5, abs=1e-7)
    assert sg == pytest.approx(o.sum_G, rel=1e-4, abs=1e-3 + 1e-6 * np.abs(o.G).sum())
    assert g.objective() == pytest.approx(o.objective, rel=1e-5)


def check_params(o, g, before):
    w0, w, V = g.get_params()
    assert np.abs(w - o.w).max() <= 1e-4 * (1 + np.abs(o.w).max())
    assert np.all(np.abs(V - o.V) <= 1e-4 * (1 + np.abs(o.V)))
    assert abs(w0 - o.w0) <= 1e-4 * (1 + abs(o.w0))
    bw0, bw, bV = before
    for got, ref, start in ((w, o.w, bw), (V, o.V, bV)):
        dref = ref - start
        dgot = got.astype(np.float64) - start
        assert np.abs(dgot - dref).max() <= 2e-3 * np.abs(dref).max() + 2e-7


@pytest.mark.parametrize("name", ["C1", "C2", "C3", "C4s", "C5s"])
def test_init_tiles_and_first_refresh(name):
    wl = W.make(name)
    o, g = make_pair(wl)
    w0, w, V = g.get_params()
    assert w0 == 0.0 and not w.any()
    assert np.array_equal(V.astype(np.float64), o.V)                      # same seeded draw, bit for bit
    tp, rows, cols, vals = g.get_tiles()
    assert np.array_equal(tp, o.tile_ptr) and np.array_equal(rows, o.rows) and np.array_equal(cols, o.cols)
    assert np.array_equal(vals.view(np.uint32), o.vals.view(np.uint32))
    check_aux(o, g)
    g.close()


@pytest.fixture(params=["rowblock", "round"])
def sweep(request, monkeypatch):
    """Launch order of the strata: one launch per row block (default) or one per inner round."""
    monkeypatch.setenv("DSFACTO_SWEEP", request.param)
    return request.param


@pytest.mark.parametrize("name,epochs", [("C1", 10), ("C2", 10), ("C3", 5), ("C4s", 2), ("C5s", 2)])
def test_epochs_match_oracle(name, epochs, sweep):
    wl = W.make(name)
    o, g = make_pair(wl)
    for e in range(epochs):
        before = (o.w0, o.w.copy(), o.V.copy())
        ref = o.epoch()
        got = g.epoch()
        assert got == pytest.approx(ref, rel=1e-4), "epoch %d" % (e + 1)
        if e == 0:
            check_params(o, g, before)
            check_aux(o, g)
    w0, w, V = g.get_params()
    assert np.abs(w - o.w).max() <= 1e-4 * (1 + np.abs(o.w).max())
    assert np.all(np.abs(V - o.V) <= 1e-4 * (1 + np.abs(o.V)))
    g.close()


def test_sensitive_case_large_step():
    # C1 data with a 200x larger step: the objective falls by a large factor in 10 epochs, so any
    # mistake in the update shows up well above the tolerance
    wl = W.make("C1")
    o, g = make_pair(wl, eta=2.0)
    start = o.objective
    for e in range(10):
        before = (o.w0, o.w.copy(), o.V.copy())
        ref, got = o.epoch(), g.epoch()
        assert got == pytest.approx(ref, rel=1e-4)
        if e in (0, 9):
            check_params(o, g, before)
    assert o.objective < 0.5 * start
    g.close()


@pytest.mark.parametrize("K", [1, 3, 4, 5, 7, 12, 20, 33, 64, 100, 128, 129, 200, 256])
def test_factor_widths(K, sweep):
    wl = W.make("C2", n=6000)
    o, g = make_pair(wl, K=K, eta=1.0, p=3)
    check_aux(o, g)
    before = (o.w0, o.w.copy(), o.V.copy())
    assert g.epoch() == pytest.approx(o.epoch(), rel=1e-4)
    check_params(o, g, before)
    g.close()


@pytest.mark.parametrize("p", [1, 2, 3, 7, 16, 100, 150, 2500])
def test_tile_grids_including_empty_blocks(p):
    # p = 150 > d = 100 leaves empty column blocks; p = 2500 > n = 2000 leaves empty row blocks too
    wl = W.make("C1")
    o, g = make_pair(wl, p=p, eta=1.0)
    tp, rows, cols, vals = g.get_tiles()
    assert np.array_equal(tp, o.tile_ptr) and np.array_equal(rows, o.rows) and np.array_equal(cols, o.cols)
    before = (o.w0, o.w.copy(), o.V.copy())
    assert g.epoch() == pytest.approx(o.epoch(), rel=1e-4)
    check_params(o, g, before)
    g.close()


def _hot_column_problem(n, d, seed):
    # column 0 is present in every row, column 1 in every second row: runs far longer than one chunk
    rng = np.random.default_rng(seed)
    rows = []
    for i in range(n):
        cols = {0}
        if i % 2 == 0:
            cols.add(1)
        cols.update(rng.choice(np.arange(2, d), size=2, replace=False).tolist())
        rows.append(sorted(cols))
    indptr = np.zeros(n + 1, np.int64)
    indptr[1:] = np.cumsum([len(r) for r in rows])
    indices = np.concatenate(rows).astype(np.int32)
    values = rng.standard_normal(len(indices)).astype(np.float32)
    y = rng.standard_normal(n).astype(np.float32)
    return indptr, indices, values, y


@pytest.mark.parametrize("K,p,loss", [(16, 1, 0), (16, 3, 1), (8, 2, 0), (128, 2, 0), (40, 1, 1)])
def test_long_runs_cross_chunk_warp_and_group_boundaries(K, p, loss, sweep):
    n, d = 9000, 12
    indptr, indices, values, y = _hot_column_problem(n, d, 3)
    if loss:
        y = np.where(y > 0, 1.0, -1.0).astype(np.float32)
    o = O.Oracle(n, d, K, p, loss, 1e-3, 1e-3, 0.5, 77)
    o.load_csr(indptr, indices, values, y)
    g = D.DSFacto(n, d, K, p, loss, 1e-3, 1e-3, 0.5, 77)
    g.load_csr(indptr, indices, values, y)
    for _ in range(3):
        before = (o.w0, o.w.copy(), o.V.copy())
        assert g.epoch() == pytest.approx(o.epoch(), rel=1e-4)
        check_params(o, g, before)
    g.close()


def test_degenerate_shapes():
    # one row; rows without entries; a column that never occurs; no stored entries at all
    cases = []
    cases.append((1, 3, np.array([0, 2], np.int64), np.array([0, 2], np.int32), np.array([1.5, -2.0], np.float32),
                  np.array([0.3], np.float32)))
    cases.append((4, 5, np.array([0, 0, 2, 2, 3], np.int64), np.array([1, 4, 0], np.int32),
                  np.array([1.0, 2.0, -1.0], np.float32), np.array([1.0, -1.0, 0.5, 0.0], np.float32)))
    cases.append((3, 4, np.array([0, 0, 0, 0], np.int64), np.zeros(0, np.int32), np.zeros(0, np.float32),
                  np.array([1.0, 2.0, 3.0], np.float32)))
    for n, d, indptr, indices, values, y in cases:
        for p in (1, 2, 5):
            o = O.Oracle(n, d, 6, p, 0, 1e-2, 1e-2, 0.3, 5)
            o.load_csr(indptr, indices, values, y)
            g = D.DSFacto(n, d, 6, p, 0, 1e-2, 1e-2, 0.3, 5)
            g.load_csr(indptr, indices, values, y)
            for _ in range(2):
                assert g.epoch() == pytest.approx(o.epoch(), rel=1e-5)
            w0, w, V = g.get_params()
            np.testing.assert_allclose(w, o.w, atol=1e-6)
            np.testing.assert_allclose(V, o.V, atol=1e-6)
            assert w0 == pytest.approx(o.w0, abs=1e-6)
            g.close()


@pytest.mark.parametrize("chunk,block", [(0, 0), (1000, 64), (2048, 192)])
def test_wide_entry_layout_on_device(monkeypatch, chunk, block):
    # local row and column need 17 bits each: entry records of {row, column} plus a value array of their own;
    # with long chunks the kernel reads both arrays block by block through its entry ring
    if chunk:
        monkeypatch.setenv("DSFACTO_CHUNK", str(chunk))
        monkeypatch.setenv("DSFACTO_BLOCK", str(block))
    n = d = 1 << 17
    indptr, indices, values, y = W.generate(n=n, d=d, seed=5, structure=W.UNIFORM, len_min=3, len_max=3,
                                            label_kind=W.L_REGRESSION, noise=0.1)
    o = O.Oracle(n, d, 4, 1, 0, 1e-3, 1e-3, 50.0, 9)
    o.load_csr(indptr, indices, values, y)
    g = D.DSFacto(n, d, 4, 1, 0, 1e-3, 1e-3, 50.0, 9)
    g.load_csr(indptr, indices, values, y)
    tp, rows, cols, vals = g.get_tiles()
    assert np.array_equal(rows, o.rows) and np.array_equal(cols, o.cols)
    before = (o.w0, o.w.copy(), o.V.copy())
    assert g.epoch() == pytest.approx(o.epoch(), rel=1e-4)
    check_params(o, g, before)
    g.close()


def test_predict_matches_oracle_scores():
    wl = W.make("C3")
    o, g = make_pair(wl)
    o.epoch(); g.epoch()
    ref = o.predict()
    got = g.predict()
    np.testing.assert_allclose(got, ref, rtol=0, atol=2e-5 * (1 + np.abs(ref).max()))
    other = W.make("C3", n=500)                                   # rows the model never saw
    ref2 = o.predict(other.indptr, other.indices, other.values)
    got2 = g.predict(other.indptr, other.indices, other.values)
    np.testing.assert_allclose(got2, ref2, rtol=0, atol=2e-5 * (1 + np.abs(ref2).max()))
    g.close()


def test_set_params_roundtrip_and_refresh():
    wl = W.make("C1")
    o, g = make_pair(wl)
    rng = np.random.default_rng(0)
    w = (rng.standard_normal(wl.d) * 0.2).astype(np.float32)
    V = (rng.standard_normal((wl.d, wl.K)) * 0.2).astype(np.float32)
    g.set_params(0.25, w, V)
    o.w0, o.w[:], o.V[:] = 0.25, w, V
    o.refresh()
    w0b, wb, Vb = g.get_params()
    assert w0b == 0.25 and np.array_equal(wb, w) and np.array_equal(Vb, V)
    check_aux(o, g)
    g.close()


def test_runs_are_bit_identical():
    wl = W.make("C3")
    outs = []
    for _ in range(2):
        g = D.DSFacto(wl.n, wl.d, wl.K, wl.p, wl.loss, wl.lambda_w, wl.lambda_v, wl.eta, wl.init_seed)
        g.load_csr(wl.indptr, wl.indices, wl.values, wl.y)
        objs = [g.epoch() for _ in range(2)]
        outs.append((objs, g.get_params()))
        g.close()
    assert outs[0][0] == outs[1][0]
    assert outs[0][1][0] == outs[1][1][0]
    assert np.array_equal(outs[0][1][1], outs[1][1][1]) and np.array_equal(outs[0][1][2], outs[1][1][2])


def test_status_codes_on_device():
    g = D.DSFacto(4, 3, 2, 2, 0, 0.0, 0.0, 0.1, 1)
    assert D.dsfacto_epoch(g._h) == D.ERR_NO_DATA
    assert D.dsfacto_objective(g._h)[0] == D.ERR_NO_DATA
    indptr = np.array([0, 1, 2, 3, 4], np.int64)
    indices = np.array([0, 1, 2, 0], np.int32)
    values = np.ones(4, np.float32)
    assert D.dsfacto_load_csr(g._h, indptr, indices, values, np.array([1, np.nan, 0, 0], np.float32)) == D.ERR_INVALID_CSR
    assert D.dsfacto_load_csr(g._h, indptr, np.array([0, 1, 3, 0], np.int32), values, np.zeros(4, np.float32)) == D.ERR_INVALID_CSR
    assert D.dsfacto_load_csr(g._h, indptr, indices, values, np.array([1, 2, 3, 4], np.float32)) == D.OK
    assert D.dsfacto_epoch(g._h) == D.OK
    g.close()
    # a step far beyond stability: the objective overflows and the call says so instead of crashing
    wl = W.make("C1")
    g = D.DSFacto(wl.n, wl.d, wl.K, wl.p, wl.loss, wl.lambda_w, wl.lambda_v, 1e6, wl.init_seed)
    g.load_csr(wl.indptr, wl.indices, wl.values, wl.y)
    rcs = [D.dsfacto_epoch(g._h) for _ in range(12)]
    assert D.ERR_DIVERGED in rcs and all(rc in (D.OK, D.ERR_DIVERGED) for rc in rcs)
    g.close()


@pytest.mark.parametrize("chunk,block", [(16, 0), (100, 0), (200, 0), (512, 0), (1000, 0), (4096, 0),
                                         (100, 32), (416, 32), (1000, 64), (2048, 256)])
@pytest.mark.parametrize("name", ["C3", "C4s", "C5s"])
def test_any_chunk_length_gives_the_same_epoch(monkeypatch, name, chunk, block):
    # the chunk length of the stratum SGD launches is a tuning parameter (DSFACTO_CHUNK overrides the
    # choice made at load time): whole passes, partial passes and chunks shorter than a pass must all
    # reproduce the oracle's epoch.  The kernel reads a chunk's entries through a ring of blocks
    # (DSFACTO_BLOCK entries each, 192 unless the chunks are shorter): chunks of one block, of a few and of
    # more blocks than the ring has slots, blocks of a single pass, a last block of a few entries.
    monkeypatch.setenv("DSFACTO_CHUNK", str(chunk))
    if block:
        monkeypatch.setenv("DSFACTO_BLOCK", str(block))
    wl = W.make(name)
    o, g = make_pair(wl)
    for _ in range(2):
        before = (o.w0, o.w.copy(), o.V.copy())
        want, got = o.epoch(), g.epoch()
        assert got == pytest.approx(want, rel=1e-4)
        check_params(o, g, before)
    g.close()
