"""Property tests of the fp64 oracle over randomly drawn small configurations (hypothesis): identities
that hold for every chunk size, k, alpha and worker count, checked against numpy / scipy rather than
against the oracle itself."""
import numpy as np
import scipy.fft
from hypothesis import given, settings
from hypothesis import strategies as st

from oracle import demo_oracle as orc

SIZES = st.sampled_from([2, 4, 8, 16, 32])


def _case(seed, s, rows_2d, n):
    rng = np.random.default_rng(seed)
    rows = s if rows_2d else 1
    M = rows * s
    return rng, rows, M, rng.standard_normal((n, M)), rng.standard_normal((n, M))


@settings(max_examples=25, deadline=None)
@given(seed=st.integers(0, 10**6), s=SIZES, rows_2d=st.booleans(), k=st.integers(1, 40), beta=st.floats(0.0, 1.0),
       alpha=st.floats(0.0, 1.0))
def test_compress_identities_hold_for_any_configuration(seed, s, rows_2d, k, beta, alpha):
    rng, rows, M, g, m = _case(seed, s, rows_2d, 3)
    out = orc.compress_chunks(g, m, s, rows, k, beta, alpha=alpha)
    k_eff = min(k, M)
    B = beta * m + g
    for c in range(3):
        # the coefficients are the library's orthonormal DCT-II of B (2-D: both axes)
        Bt = B[c].reshape(rows, s)
        Qw = scipy.fft.dctn(Bt, type=2, norm="ortho") if rows > 1 else scipy.fft.dct(Bt[0], type=2, norm="ortho")
        assert np.max(np.abs(out["Q"][c] - Qw.reshape(-1))) < 1e-11 * max(1.0, np.max(np.abs(Qw)))
        # the kept set: k_eff distinct ascending indices, every kept magnitude >= every dropped one
        idx = out["idx"][c]
        assert idx.shape == (k_eff,) and np.all(np.diff(idx) > 0) and idx[0] >= 0 and idx[-1] < M
        mag = np.abs(out["Q"][c])
        dropped = np.setdiff1d(np.arange(M), idx)
        if dropped.size:
            assert mag[idx].min() >= mag[dropped].max()
        assert np.array_equal(out["val"][c], out["Q"][c][idx])
        # residual: B minus alpha times the inverse transform of the kept coefficients
        Qs = np.zeros(M)
        Qs[idx] = out["val"][c]
        Qs = Qs.reshape(rows, s)
        back = scipy.fft.idctn(Qs, type=2, norm="ortho") if rows > 1 else scipy.fft.idct(Qs[0], type=2, norm="ortho")
        assert np.max(np.abs(out["m_new"][c] - (B[c] - alpha * back.reshape(-1)))) < 1e-11 * max(1.0, np.max(np.abs(B[c])))


@settings(max_examples=25, deadline=None)
@given(seed=st.integers(0, 10**6), s=SIZES, rows_2d=st.booleans(), k=st.integers(1, 12), W=st.integers(1, 5),
       agg=st.sampled_from([orc.AGG_SUM, orc.AGG_MEAN, orc.AGG_COUNT_MEAN]), phi=st.sampled_from([orc.PHI_SIGN, orc.PHI_IDENTITY]))
def test_decode_matches_a_direct_numpy_evaluation(seed, s, rows_2d, k, W, agg, phi):
    rng, rows, M, _, _ = _case(seed, s, rows_2d, 2)
    k_eff = min(k, M)
    recs = np.zeros((W, 2, k_eff), dtype=orc.RECORD_DTYPE)
    for w in range(W):
        for c in range(2):
            recs[w, c]["idx"] = np.sort(rng.choice(M, size=k_eff, replace=False))
            recs[w, c]["val"] = rng.standard_normal(k_eff).astype(np.float32)
    x = rng.standard_normal((2, M)) * 0.02
    lr, wd = 1e-3, 0.1
    out = orc.decode_chunks(recs, x, s, rows, lr, wd, agg=agg, phi=phi)
    for c in range(2):
        S = np.zeros(M)
        cnt = np.zeros(M)
        for w in range(W):
            np.add.at(S, recs[w, c]["idx"], recs[w, c]["val"].astype(np.float64))
            np.add.at(cnt, recs[w, c]["idx"], 1.0)
        if agg == orc.AGG_MEAN:
            S = S / W
        elif agg == orc.AGG_COUNT_MEAN:
            S = np.where(cnt > 0, S / np.maximum(cnt, 1.0), 0.0)
        St = S.reshape(rows, s)
        R = scipy.fft.idctn(St, type=2, norm="ortho") if rows > 1 else scipy.fft.idct(St[0], type=2, norm="ortho")
        R = R.reshape(-1)
        assert np.max(np.abs(out["R"][c] - R)) < 1e-12 * max(1.0, np.max(np.abs(R)))
        upd = np.sign(out["R"][c]) if phi == orc.PHI_SIGN else out["R"][c]
        assert np.max(np.abs(out["x_new"][c] - (x[c] - lr * (upd + wd * x[c])))) < 1e-16
