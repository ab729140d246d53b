"""dsfacto_score_loss_noalloc against the ordinary entry points.

The allocation-free call exists for hosts that may not call cudaMalloc while they work (all device
memory belongs to someone else's pool, or the thread must not touch the driver's allocator).  It
keeps its reduction scratch in a fixed array inside the library, shared by every call, so this test
runs it twice in a row on different inputs: the second result must not be coloured by what the
first call left behind.  Reference values come from the handle-based path (dsfacto_predict for the
scores, dsfacto_get_stats for the two sums), with the tolerances the other GPU tests use, and the
scores and the loss sum are also held against the CPU oracle's own evaluation of the same rows.

The file name sorts last on purpose: if this extra entry point breaks, a run that stops at the
first failure has already gone through every other test."""
import numpy as np
import pytest

from oracle import dsfacto_oracle as O
from paper_2004_13940_b200 import dsfacto as D
from paper_2004_13940_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _reference(wl, w0, w, V):
    g = D.DSFacto(wl.n, wl.d, wl.K, wl.p, wl.loss, wl.lambda_w, wl.lambda_v, wl.eta, wl.init_seed)
    g.load_csr(wl.indptr, wl.indices, wl.values, wl.y)
    g.set_params(w0, w, V)
    scores = g.predict()
    mean_loss, sum_g = g.stats()
    g.close()
    return scores, mean_loss * wl.n, sum_g


def _no_alloc(wl, w0, w, V):
    import torch

    dev = torch.device("cuda", 0)
    t = {k: torch.from_numpy(np.ascontiguousarray(a)).to(dev) for k, a in
         dict(indptr=wl.indptr, indices=wl.indices, values=wl.values, y=wl.y, w=w, V=V).items()}
    scores = torch.empty(wl.n, dtype=torch.float32, device=dev)
    sums = torch.full((2,), float("nan"), dtype=torch.float64, device=dev)
    torch.cuda.synchronize()
    rc = D.dsfacto_score_loss_noalloc(wl.n, wl.d, wl.K, wl.loss, t["indptr"].data_ptr(), t["indices"].data_ptr(),
                                      t["values"].data_ptr(), t["y"].data_ptr(), w0, t["w"].data_ptr(),
                                      t["V"].data_ptr(), scores.data_ptr(), sums.data_ptr(), 0)
    assert rc == D.OK
    return scores.cpu().numpy(), float(sums[0]), float(sums[1])


def _check(wl, seed):
    rng = np.random.default_rng(seed)
    w0 = float(np.float32(rng.standard_normal() * 0.1))
    w = (rng.standard_normal(wl.d) * 0.1).astype(np.float32)
    V = (rng.standard_normal((wl.d, wl.K)) * 0.1).astype(np.float32)
    ref_scores, ref_loss, ref_g = _reference(wl, w0, w, V)
    scores, loss_sum, g_sum = _no_alloc(wl, w0, w, V)
    np.testing.assert_allclose(scores, ref_scores, rtol=0, atol=2e-5 * (1 + np.abs(ref_scores).max()))
    assert loss_sum == pytest.approx(ref_loss, rel=1e-5, abs=1e-6)
    assert g_sum == pytest.approx(ref_g, rel=1e-4, abs=1e-3)
    # the oracle: scores by eq. (fm_model2) in fp64, mean loss over the same rows
    w64, V64 = w.astype(np.float64), V.astype(np.float64)
    want = O.score(wl.indptr, wl.indices, wl.values, w0, w64, V64)
    np.testing.assert_allclose(scores, want, rtol=0, atol=2e-5 * (1 + np.abs(want).max()))
    mean_loss, _ = O.evaluate(wl.loss, wl.indptr, wl.indices, wl.values, wl.y, w0, w64, V64)
    assert loss_sum == pytest.approx(mean_loss * wl.n, rel=1e-4)


def test_two_calls_in_a_row_match_the_handle_based_path():
    # a larger logistic problem first, a smaller squared-loss one second: the second call uses
    # fewer scratch slots than the first left filled
    _check(W.make("C3"), seed=1)          # 72,000 rows, K = 32, logistic
    _check(W.make("C1"), seed=2)          # 2,000 rows, K = 8, squared


@pytest.mark.parametrize("K", [4, 256])
def test_narrowest_and_widest_factor_rows(K):
    # K = 4 is one lane per row, K = 256 two 16-byte pieces per lane of a whole warp: the two ends of the
    # lane layouts the entry point is built for
    wl = W.make("C2", n=3000)
    wl.K = K
    _check(wl, seed=K)
    _check(wl, seed=K + 1)


def test_limits_are_rejected_with_a_clear_status():
    import torch

    buf = torch.zeros(64, dtype=torch.float64, device="cuda")
    p = buf.data_ptr()
    ok_args = dict(m=4, d=4, K=8, loss=0)

    def call(**kw):
        a = dict(ok_args); a.update(kw)
        return D.dsfacto_score_loss_noalloc(a["m"], a["d"], a["K"], a["loss"], p, p, p, p, 0.0, p, p, p, p, 0)

    assert call(K=12) == D.ERR_INVALID_ARG                    # not a whole power-of-two lane group
    assert call(K=512) == D.ERR_INVALID_ARG
    assert call(m=67_108_865) == D.ERR_INVALID_ARG            # beyond the fixed scratch array
    assert call(m=0) == D.ERR_INVALID_ARG
    assert call(loss=3) == D.ERR_INVALID_ARG
    # V not 16-byte aligned: refused on the host, never handed to the kernel
    assert D.dsfacto_score_loss_noalloc(4, 4, 8, 0, p, p, p, p, 0.0, p, p + 4, p, p, 0) == D.ERR_INVALID_ARG
    assert D.lib().dsfacto_score_loss_noalloc(4, 4, 8, 0, None, None, None, None, 0.0, None, None, None, None,
                                              None) == D.ERR_INVALID_ARG
