"""The ways dsfacto_load_csr builds the tile lists on the device give the same lists, bit for bit, as the
oracle's bucketing: the plain host bucketer, the row-block bucketer, the streamed load (row blocks
bucketed into page-locked staging memory and copied block by block; DSFACTO_LOAD=stream forces it on small
loads), and the bucketing on the device itself (keys, a stable radix sort, the chunk plan cut by a kernel),
which loads take by default when the packed entry layout applies (DSFACTO_LOAD=device asks for it by name).  DSFACTO_LOAD=nostaging
makes the streamed load behave as if no page-locked memory could be had, which must end in the row-block
bucketer with one copy, not in an error."""
import numpy as np
import pytest

from oracle import dsfacto_oracle as O
from paper_2004_13940_b200 import dsfacto as D
from paper_2004_13940_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("mode", ["device", "stream", "nostaging", "simple", None])
@pytest.mark.parametrize("name,kw", [("C3", {}), ("C4s", {}), ("C4s", {"p": 200}), ("C5s", {"p": 64}), ("C2", {"p": 40}),
                                     ("C1", {"p": 2500})])
def test_load_paths_give_the_oracle_tiles_and_epochs(monkeypatch, mode, name, kw):
    if mode is None:
        monkeypatch.delenv("DSFACTO_LOAD", raising=False)
    else:
        monkeypatch.setenv("DSFACTO_LOAD", mode)
    wl = W.make(name, **kw)
    o = O.Oracle(wl.n, wl.d, wl.K, wl.p, wl.loss, wl.lambda_w, wl.lambda_v, wl.eta, wl.init_seed)
    o.load_csr(wl.indptr, wl.indices, wl.values, wl.y)
    with D.DSFacto(wl.n, wl.d, wl.K, wl.p, wl.loss, wl.lambda_w, wl.lambda_v, wl.eta, wl.init_seed) as g:
        g.load_csr(wl.indptr, wl.indices, wl.values, wl.y)
        tp, rows, cols, vals = g.get_tiles()
        assert np.array_equal(tp, o.tile_ptr)
        assert np.array_equal(rows, o.rows) and np.array_equal(cols, o.cols) and np.array_equal(vals, o.vals)
        want, got = o.epoch(), g.epoch()
        assert got == pytest.approx(want, rel=1e-4)
        # a second load on the same handle (staging memory is reused) replaces the data set
        g.load_csr(wl.indptr, wl.indices, wl.values, wl.y)
        tp2, rows2, cols2, vals2 = g.get_tiles()
        assert np.array_equal(tp2, tp) and np.array_equal(rows2, rows) and np.array_equal(cols2, cols)


def test_streamed_load_of_the_wide_entry_layout(monkeypatch):
    # 2^16 rows x 2^17 columns per tile: local ids need 33 bits, so entries travel as {row, column} + value
    monkeypatch.setenv("DSFACTO_LOAD", "stream")
    rng = np.random.default_rng(5)
    n, d, p, K = 1 << 21, 1 << 22, 32, 4
    per_row = 3
    indices = np.sort(rng.integers(0, d, size=(n, per_row)), axis=1).astype(np.int32)
    keep = np.ones_like(indices, bool)
    keep[:, 1:] = indices[:, 1:] != indices[:, :-1]
    indptr = np.concatenate([[0], np.cumsum(keep.sum(1))]).astype(np.int64)
    idx = indices[keep]
    vals = rng.standard_normal(idx.shape[0]).astype(np.float32)
    y = rng.standard_normal(n).astype(np.float32)
    o = O.Oracle(n, d, K, p, O.SQUARED, 1e-3, 1e-3, 0.01, 7)
    o.load_csr(indptr, idx, vals, y)
    with D.DSFacto(n, d, K, p, D.SQUARED, 1e-3, 1e-3, 0.01, 7) as g:
        g.load_csr(indptr, idx, vals, y)
        tp, rows, cols, v = g.get_tiles()
        assert np.array_equal(tp, o.tile_ptr) and np.array_equal(rows, o.rows) and np.array_equal(cols, o.cols)
        assert np.array_equal(v, o.vals)
        assert g.epoch() == pytest.approx(o.epoch(), rel=1e-4)


@pytest.mark.parametrize("sweep", [None, "round"])
@pytest.mark.parametrize("name,kw", [("C1", {}), ("C2", {}), ("C3", {}), ("C4s", {}), ("C5s", {}), ("C3", {"p": 7})])
def test_device_bucketing_gives_the_same_bits_as_the_host(monkeypatch, sweep, name, kw):
    # same tile lists and the same chunk plan, hence the same parameters bit for bit; also with rows and
    # columns emptied so that tiles, rows and whole column blocks are empty
    if sweep:
        monkeypatch.setenv("DSFACTO_SWEEP", sweep)
    else:
        monkeypatch.delenv("DSFACTO_SWEEP", raising=False)
    wl = W.make(name, **kw)
    keep = np.ones(wl.indices.shape[0], bool)
    rows = np.repeat(np.arange(wl.n), np.diff(wl.indptr))
    keep[(rows % 7) == 3] = False                       # every seventh row empty
    keep[(wl.indices * wl.p) // wl.d == wl.p // 2] = False   # one column block empty
    indptr = np.concatenate([[0], np.cumsum(np.bincount(rows[keep], minlength=wl.n))]).astype(np.int64)
    indices, values = wl.indices[keep], wl.values[keep]
    res = []
    monkeypatch.setenv("DSFACTO_ROW_MERGE", "1")   # (slots of several row blocks, which only the device builds, round differently)
    for mode in ("device", "simple"):
        monkeypatch.setenv("DSFACTO_LOAD", mode)
        with D.DSFacto(wl.n, wl.d, wl.K, wl.p, wl.loss, wl.lambda_w, wl.lambda_v, wl.eta, wl.init_seed) as g:
            g.load_csr(indptr, indices, values, wl.y)
            tiles = g.get_tiles()
            objs = [g.objective()] + [g.epoch() for _ in range(2)]
            w0, w, V = g.get_params()
        res.append((tiles, objs, w0, w, V))
    for a, b in zip(res[0][0], res[1][0]):
        assert np.array_equal(a, b)
    assert res[0][1] == res[1][1] and res[0][2] == res[1][2]
    assert np.array_equal(res[0][3], res[1][3]) and np.array_equal(res[0][4], res[1][4])


def test_a_rejected_large_load_leaves_the_handle_as_it_was():
    # from 2^24 entries on the CSR arrays travel to the device while the host still checks them; a data set
    # that fails the checks must not replace the one the handle holds
    wl = W.make("C4", n=600_000, p=64)
    assert wl.nnz >= 1 << 24
    with D.DSFacto(wl.n, wl.d, wl.K, wl.p, wl.loss, wl.lambda_w, wl.lambda_v, wl.eta, wl.init_seed) as g, \
            D.DSFacto(wl.n, wl.d, wl.K, wl.p, wl.loss, wl.lambda_w, wl.lambda_v, wl.eta, wl.init_seed) as ref:
        g.load_csr(wl.indptr, wl.indices, wl.values, wl.y)
        ref.load_csr(wl.indptr, wl.indices, wl.values, wl.y)
        assert g.last_load()[0] == 2          # bucketed on the device
        obj0 = g.objective()
        bad_idx = wl.indices.copy()
        r = wl.n // 2
        b = wl.indptr[r]
        bad_idx[b], bad_idx[b + 1] = bad_idx[b + 1], bad_idx[b]          # one row out of order
        assert D.dsfacto_load_csr(g._h, wl.indptr, bad_idx, wl.values, wl.y) == D.ERR_INVALID_CSR
        bad_val = wl.values.copy()
        bad_val[-1] = np.nan
        assert D.dsfacto_load_csr(g._h, wl.indptr, wl.indices, bad_val, wl.y) == D.ERR_INVALID_CSR
        bad_ptr = wl.indptr.copy()
        bad_ptr[5] = bad_ptr[6] + 1                                      # row pointers not monotone
        assert D.dsfacto_load_csr(g._h, bad_ptr, wl.indices, wl.values, wl.y) == D.ERR_INVALID_CSR
        assert g.objective() == obj0
        assert g.epoch() == ref.epoch()
        w0a, wa, Va = g.get_params()
        w0b, wb, Vb = ref.get_params()
        assert w0a == w0b and np.array_equal(wa, wb) and np.array_equal(Va, Vb)


@pytest.mark.parametrize("merge", [2, 4, 8, 16])
@pytest.mark.parametrize("name,kw", [("C1", {"p": 16}), ("C2", {}), ("C3", {}), ("C3", {"p": 7}), ("C4s", {}), ("C5s", {})])
def test_merged_row_blocks_on_the_device(monkeypatch, merge, name, kw):
    # Several row blocks per slot: a column's entries of consecutive row blocks are stored and swept as one
    # run.  The canonical tile lists that come back are still the oracle's, bit for bit; the epochs are the
    # oracle's within the tolerance (runs are cut elsewhere, so the bits differ from the one-tile-per-slot plan).
    monkeypatch.setenv("DSFACTO_LOAD", "device")
    monkeypatch.delenv("DSFACTO_SWEEP", raising=False)
    wl = W.make(name, **kw)
    keep = np.ones(wl.indices.shape[0], bool)
    rows = np.repeat(np.arange(wl.n), np.diff(wl.indptr))
    keep[(rows % 11) == 5] = False                       # some rows empty
    indptr = np.concatenate([[0], np.cumsum(np.bincount(rows[keep], minlength=wl.n))]).astype(np.int64)
    indices, values = wl.indices[keep], wl.values[keep]
    o = O.Oracle(wl.n, wl.d, wl.K, wl.p, wl.loss, wl.lambda_w, wl.lambda_v, wl.eta, wl.init_seed)
    o.load_csr(indptr, indices, values, wl.y)
    with D.DSFacto(wl.n, wl.d, wl.K, wl.p, wl.loss, wl.lambda_w, wl.lambda_v, wl.eta, wl.init_seed) as g:
        g.debug_set(D.DEBUG_ROW_MERGE, merge)
        g.load_csr(indptr, indices, values, wl.y)
        assert g.last_load()[0] == 2
        tp, r, c, v = g.get_tiles()
        assert np.array_equal(tp, o.tile_ptr)
        assert np.array_equal(r, o.rows) and np.array_equal(c, o.cols) and np.array_equal(v, o.vals)
        assert g.objective() == pytest.approx(o.objective, rel=1e-5)
        for _ in range(3):
            assert g.epoch() == pytest.approx(o.epoch(), rel=1e-4)
        w0, w, V = g.get_params()
        A, G = g.get_aux()
        # the same epochs again on a second handle: the same bits
        with D.DSFacto(wl.n, wl.d, wl.K, wl.p, wl.loss, wl.lambda_w, wl.lambda_v, wl.eta, wl.init_seed) as g2:
            g2.debug_set(D.DEBUG_ROW_MERGE, merge)
            g2.load_csr(indptr, indices, values, wl.y)
            for _ in range(3):
                g2.epoch()
            w0b, wb, Vb = g2.get_params()
    assert w0 == w0b and np.array_equal(w, wb) and np.array_equal(V, Vb)
    assert abs(w0 - o.w0) <= 1e-4 * (1 + abs(o.w0))
    assert np.abs(w - o.w).max() <= 1e-4 * (1 + np.abs(o.w).max())
    assert np.all(np.abs(V - o.V) <= 1e-4 * (1 + np.abs(o.V)))
    assert np.all(np.abs(G - o.G) <= 1e-4 * (1 + np.abs(o.G)))
