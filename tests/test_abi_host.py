"""CPU-side checks of the CUDA library: it loads, exports every symbol the header declares, and
its host logic (argument checks, CSR validation, the tile bucketer) behaves.  No kernel runs."""
import re
from pathlib import Path

import numpy as np
import pytest

from oracle import dsfacto_oracle as O
from paper_2004_13940_b200 import dsfacto as D
from paper_2004_13940_b200 import workloads as W
from tests.helpers import tiny_problem

HEADER = Path(__file__).resolve().parent.parent / "include" / "dsfacto.h"


def declared_functions():
    text = re.sub(r"/\*.*?\*/", "", HEADER.read_text(), flags=re.S)
    return sorted(set(re.findall(r"\b(dsfacto_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = declared_functions()
    assert "dsfacto_create" in names and "dsfacto_epoch" in names and len(names) >= 12
    L = D.lib()
    for name in names:
        assert hasattr(L, name), name
    assert sorted(D.SIGNATURES) == names          # the binding covers exactly the header


def test_strerror_and_argument_checks():
    L = D.lib()
    assert L.dsfacto_strerror(0) == b"ok"
    assert b"CSR" in L.dsfacto_strerror(D.ERR_INVALID_CSR)
    for bad in (dict(n=0), dict(d=0), dict(K=0), dict(K=257), dict(p=0), dict(loss=2), dict(eta=0.0),
                dict(lambda_w=-1.0)):
        kw = dict(n=10, d=5, K=4, p=2, loss=0, lambda_w=0.0, lambda_v=0.0, eta=0.1, seed=1)
        kw.update(bad)
        rc, h = D.dsfacto_create(**kw)
        assert rc == D.ERR_INVALID_ARG and not h.value


def test_create_without_device_fails_loudly():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    rc, h = D.dsfacto_create(10, 5, 4, 2, 0, 0.0, 0.0, 0.1, 1)
    assert rc == D.ERR_CUDA and not h.value
    with pytest.raises(D.DSFactoError):
        D.DSFacto(10, 5, 4, 2, 0, 0.0, 0.0, 0.1, 1)


@pytest.mark.parametrize("n,d,p,density", [(40, 30, 4, 0.3), (17, 5, 3, 0.7), (9, 3, 5, 0.9), (25, 11, 1, 0.4),
                                           (6, 40, 6, 0.2), (3, 2, 7, 1.0)])
def test_host_bucketer_bit_exact_vs_oracle_small(n, d, p, density):
    rng = np.random.default_rng(n + 31 * d)
    _, _, indptr, indices, vals, *_ = tiny_problem(rng, n, d, 2, density)
    rc, tp, rows, cols, tv = D.dsfacto_bucket_host(n, d, p, indptr, indices, vals)
    assert rc == D.OK
    otp, orows, ocols, ovals = O.bucket(n, d, p, indptr, indices, vals)
    assert np.array_equal(tp, otp) and np.array_equal(rows, orows) and np.array_equal(cols, ocols)
    assert np.array_equal(tv.view(np.uint32), ovals.view(np.uint32))


@pytest.mark.parametrize("name,kw", [("C1", {}), ("C2", {}), ("C3", {}), ("C4s", {}), ("C5s", {}),
                                     ("C4", dict(n=300_000, p=512)), ("C1", dict(p=1)), ("C2", dict(p=64))])
def test_host_bucketer_bit_exact_vs_oracle_workloads(name, kw):
    wl = W.make(name, **kw)
    rc, tp, rows, cols, tv = D.dsfacto_bucket_host(wl.n, wl.d, wl.p, wl.indptr, wl.indices, wl.values)
    assert rc == D.OK
    otp, orows, ocols, ovals = O.bucket(wl.n, wl.d, wl.p, wl.indptr, wl.indices, wl.values)
    assert np.array_equal(tp, otp)
    assert np.array_equal(rows, orows) and np.array_equal(cols, ocols)
    assert np.array_equal(tv.view(np.uint32), ovals.view(np.uint32))


def test_wide_entry_layout_when_local_ids_exceed_32_bits():
    # p = 1 with 2^17 rows and 2^17 columns needs 34 bits of local ids -> unpacked entries
    n = d = 1 << 17
    indptr, indices, values, y = W.generate(n=n, d=d, seed=5, structure=W.UNIFORM, len_min=3, len_max=3)
    rc, tp, rows, cols, tv = D.dsfacto_bucket_host(n, d, 1, indptr, indices, values)
    assert rc == D.OK
    otp, orows, ocols, ovals = O.bucket(n, d, 1, indptr, indices, values)
    assert np.array_equal(tp, otp) and np.array_equal(rows, orows) and np.array_equal(cols, ocols)
    assert np.array_equal(tv, ovals)


def test_csr_validation_rejects_malformed_input():
    indptr = np.array([0, 2, 4], np.int64)
    good = np.array([0, 2, 1, 3], np.int32)
    vals = np.ones(4, np.float32)
    ok = lambda ip, ix, v: D.dsfacto_bucket_host(2, 4, 2, ip, ix, v)[0]
    assert ok(indptr, good, vals) == D.OK
    assert ok(indptr, np.array([2, 0, 1, 3], np.int32), vals) == D.ERR_INVALID_CSR      # unsorted
    assert ok(indptr, np.array([0, 0, 1, 3], np.int32), vals) == D.ERR_INVALID_CSR      # duplicate
    assert ok(indptr, np.array([0, 4, 1, 3], np.int32), vals) == D.ERR_INVALID_CSR      # out of range
    assert ok(indptr, np.array([-1, 2, 1, 3], np.int32), vals) == D.ERR_INVALID_CSR     # negative
    assert ok(indptr, good, np.array([1, np.nan, 1, 1], np.float32)) == D.ERR_INVALID_CSR
    assert ok(indptr, good, np.array([1, np.inf, 1, 1], np.float32)) == D.ERR_INVALID_CSR
    assert ok(np.array([0, 3, 2], np.int64), good, vals) == D.ERR_INVALID_CSR           # not monotone
    assert ok(np.array([1, 2, 4], np.int64), good, vals) == D.ERR_INVALID_CSR           # indptr[0] != 0
    assert ok(indptr, good, np.array([0, 1, 1, 1], np.float32)) == D.OK                 # stored zero is legal
