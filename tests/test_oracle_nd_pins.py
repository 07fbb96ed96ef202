"""Pins of the d-dimensional / rectangular-chunk oracle against things other than itself: the
definitions of the paper's appendix written as brute-force loops, the paper's worked blocking example,
scipy's DCT, closed forms, and the separately written C oracle on the cases both cover."""
import itertools

import numpy as np
import pytest
import scipy.fft

from oracle import demo_oracle as orc
from oracle import demo_oracle_nd as ond


def test_dct_matrix_values_and_orthonormality():
    # textbook values: s = 2 is [[1, 1], [1, -1]] / sqrt(2); s = 4 row 1; s = 3 closed form
    np.testing.assert_allclose(ond.dct_matrix(2), np.array([[1, 1], [1, -1]]) / np.sqrt(2), atol=1e-15)
    np.testing.assert_allclose(ond.dct_matrix(4)[1], [0.6532814824, 0.2705980501, -0.2705980501, -0.6532814824],
                               atol=1e-9)
    np.testing.assert_allclose(ond.dct_matrix(3)[1], [np.sqrt(2 / 3) * np.cos(np.pi / 6), 0.0,
                                                      -np.sqrt(2 / 3) * np.cos(np.pi / 6)], atol=1e-15)
    for s in (1, 3, 5, 12, 24, 48, 96, 128):
        C = ond.dct_matrix(s)
        assert np.max(np.abs(C @ C.T - np.eye(s))) < 1e-12
        np.testing.assert_allclose(C, orc.dct_matrix(s), atol=1e-15)  # the C oracle's closed form


def test_multilinear_is_the_definition_by_brute_force():
    """The multilinear product of the appendix as d nested sums, with matrices that are not orthogonal
    (a transposed or swapped operand would show)."""
    rng = np.random.default_rng(0)
    for shape in ((2, 3, 4), (3, 2), (4,), (2, 2, 3, 2)):
        X = rng.standard_normal(shape)
        Ps = [rng.standard_normal((s, s)) for s in shape]
        want = np.zeros(shape)
        for i in itertools.product(*[range(s) for s in shape]):
            acc = 0.0
            for j in itertools.product(*[range(s) for s in shape]):
                w = 1.0
                for ax in range(len(shape)):
                    w *= Ps[ax][i[ax], j[ax]]
                acc += w * X[j]
            want[i] = acc
        np.testing.assert_allclose(ond.multilinear(X, Ps), want, rtol=1e-12, atol=1e-12)


def test_multilinear_order_two_is_the_matrix_form():
    rng = np.random.default_rng(1)
    X = rng.standard_normal((5, 7))
    P0, P1 = rng.standard_normal((5, 5)), rng.standard_normal((7, 7))
    np.testing.assert_allclose(ond.multilinear(X, [P0, P1]), P0 @ X @ P1.T, rtol=1e-12, atol=1e-12)


def test_blocking_example_of_the_paper():
    """Appendix example: a 128 x 512 matrix in 16 x 32 blocks gives an 8 x 16 grid with
    B_{k0,k1}[j0][j1] = X[16 k0 + j0][32 k1 + j1]."""
    X = np.arange(128 * 512, dtype=np.float64).reshape(128, 512)
    Bk = ond.blocks(X, (16, 32))
    assert Bk.shape == (8, 16, 16, 32)
    for k0, k1, j0, j1 in ((0, 0, 0, 0), (0, 0, 15, 31), (7, 15, 15, 31), (3, 9, 4, 17), (5, 0, 0, 31)):
        assert Bk[k0, k1, j0, j1] == X[16 * k0 + j0, 32 * k1 + j1]
    np.testing.assert_array_equal(Bk[0, 0], X[:16, :32])
    np.testing.assert_array_equal(ond.unblocks(Bk, X.shape), X)
    np.testing.assert_array_equal(Bk[2, 5], orc.block_extract(X, 16, 32, 2, 5))  # the C oracle's indexer


def test_blocking_order_three_by_index_formula():
    shape, chunk = (4, 6, 10), (2, 3, 5)
    X = np.arange(np.prod(shape), dtype=np.float64).reshape(shape)
    Bk = ond.blocks(X, chunk)
    assert Bk.shape == (2, 2, 2, 2, 3, 5)
    for k in itertools.product(range(2), range(2), range(2)):
        for j in itertools.product(range(2), range(3), range(5)):
            assert Bk[k + j] == X[tuple(k[a] * chunk[a] + j[a] for a in range(3))]
    np.testing.assert_array_equal(ond.unblocks(Bk, shape), X)
    with pytest.raises(ValueError):
        ond.blocks(X, (3, 3, 5))


@pytest.mark.parametrize("chunk", [(16, 32), (8, 4, 6), (3, 5), (12,), (2, 4, 2, 8)])
def test_chunk_transform_is_scipy_dctn(chunk):
    """With the DCT matrices the multilinear product is the orthonormal d-dimensional DCT-II."""
    rng = np.random.default_rng(2)
    B = rng.standard_normal(chunk)
    Cs = [ond.dct_matrix(s) for s in chunk]
    Q = ond.multilinear(B, Cs)
    np.testing.assert_allclose(Q, scipy.fft.dctn(B, type=2, norm="ortho"), rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(ond.multilinear(Q, [C.T for C in Cs]), B, rtol=1e-11, atol=1e-12)
    assert abs(np.sum(Q * Q) - np.sum(B * B)) < 1e-11 * np.sum(B * B)  # unitary: energy is kept
    # a constant chunk has one coefficient: a * sqrt(M)
    Qc = ond.multilinear(np.full(chunk, 0.25), Cs)
    assert abs(Qc.reshape(-1)[0] - 0.25 * np.sqrt(np.prod(chunk))) < 1e-12
    assert np.max(np.abs(Qc.reshape(-1)[1:])) < 1e-13


def test_topk_is_the_stable_sort_and_breaks_ties_low():
    q = np.array([0.5, -2.0, 2.0, 0.5, -0.5, 3.0, 0.0])
    sel, a_k, a_k1 = ond.topk(q, 4)
    np.testing.assert_array_equal(sel, [0, 1, 2, 5])  # |0.5| three times: index 0 wins
    assert (a_k, a_k1) == (0.5, 0.5)
    sel, a_k, a_k1 = ond.topk(q, 100)
    np.testing.assert_array_equal(sel, np.arange(7))
    rng = np.random.default_rng(3)
    for _ in range(20):
        v = rng.standard_normal(60).round(1)  # many ties
        k = int(rng.integers(1, 60))
        want = sorted(sorted(range(60), key=lambda i: (-abs(v[i]), i))[:k])
        np.testing.assert_array_equal(ond.topk(v, k)[0], want)
        np.testing.assert_array_equal(ond.topk(v, k)[0], orc.topk(v, k)[0])


def test_square_and_one_dimensional_cases_equal_the_c_oracle():
    """Where both oracles apply (s x s tiles, length-s segments) they were written separately and must
    agree: records bit for bit, residual and decode to rounding."""
    rng = np.random.default_rng(4)
    for shape, s, k in (((32, 48), 16, 9), ((64,), 8, 3), ((16, 16), 8, 64)):
        g = rng.standard_normal(shape).astype(np.float32)
        m = rng.standard_normal(shape).astype(np.float32)
        chunk = (s,) * len(shape)
        for alpha in (1.0, 0.25):
            a = ond.compress_tensor(g, m, chunk, k, 0.9, alpha=alpha)
            b = orc.compress_tensor(g, m, s, k, 0.9, alpha=alpha)
            np.testing.assert_array_equal(a["records"]["idx"], b["records"]["idx"])
            np.testing.assert_array_equal(a["records"]["val"], b["records"]["val"])
            np.testing.assert_allclose(a["m_new"], b["m_new"], rtol=0, atol=1e-13)
            np.testing.assert_allclose(a["gap"], b["gap"], rtol=0, atol=1e-13)
        x = rng.standard_normal(shape).astype(np.float32)
        pay = [ond.compress_tensor(rng.standard_normal(shape), m, chunk, k, 0.9)["records"] for _ in range(3)]
        for agg in (0, 1, 2):
            for phi in (0, 1):
                a = ond.decode_tensor(pay, x, chunk, 1e-2, 0.1, agg=agg, phi=phi)
                b = orc.decode_tensor(pay, x, s, k, 1e-2, 0.1, agg=agg, phi=phi)
                np.testing.assert_allclose(a["R"], b["R"], rtol=0, atol=1e-13)
                np.testing.assert_allclose(a["x_new"], b["x_new"], rtol=0, atol=1e-14)


@pytest.mark.parametrize("shape,chunk,k", [((32, 96), (16, 32), 20), ((8, 6, 10), (4, 3, 5), 7),
                                             ((4, 4, 6, 8), (2, 2, 3, 4), 5), ((24, 10), (3, 5), 4)])
def test_residual_identities(shape, chunk, k):
    """DCT(m_new) vanishes on the kept set and equals Q elsewhere; IDCT(records) + m_new = beta m + g;
    the energy splits; k = M is lossless."""
    rng = np.random.default_rng(5)
    g, m = rng.standard_normal(shape), rng.standard_normal(shape)
    beta = 0.95
    M = int(np.prod(chunk))
    out = ond.compress_tensor(g, m, chunk, k, beta)
    Cs = [ond.dct_matrix(s) for s in chunk]
    Bb = ond.blocks(beta * m + g, chunk).reshape(-1, *chunk)
    Rb = ond.blocks(out["m_new"], chunk).reshape(-1, *chunk)
    for c in range(Bb.shape[0]):
        Q = scipy.fft.dctn(Bb[c], norm="ortho").reshape(-1)
        Qr = scipy.fft.dctn(Rb[c], norm="ortho").reshape(-1)
        idx = out["records"]["idx"][c]
        assert len(idx) == k and np.all(np.diff(idx) > 0)
        keep = np.zeros(M, bool)
        keep[idx] = True
        assert np.max(np.abs(Qr[keep])) < 1e-12
        np.testing.assert_allclose(Qr[~keep], Q[~keep], atol=1e-12)
        assert np.abs(Q[keep]).min() >= np.abs(Q[~keep]).max()
        np.testing.assert_allclose(out["val64"][c], Q[idx], atol=1e-12)
        assert abs(np.sum(Rb[c] ** 2) - (np.sum(Q ** 2) - np.sum(Q[keep] ** 2))) < 1e-10
        sparse = np.zeros(M)
        sparse[idx] = out["val64"][c]
        np.testing.assert_allclose(scipy.fft.idctn(sparse.reshape(chunk), norm="ortho") + Rb[c], Bb[c], atol=1e-12)
    full = ond.compress_tensor(g, m, chunk, M, beta)
    assert np.max(np.abs(full["m_new"])) < 1e-12
    # alpha scales the removed part: m_new(alpha) = B - alpha (B - m_new(1)); alpha = 0 leaves B
    half = ond.compress_tensor(g, m, chunk, k, beta, alpha=0.5)
    np.testing.assert_allclose(half["m_new"], (beta * m + g) - 0.5 * ((beta * m + g) - out["m_new"]), atol=1e-12)
    np.testing.assert_array_equal(half["records"], out["records"])
    np.testing.assert_allclose(ond.compress_tensor(g, m, chunk, k, beta, alpha=0.0)["m_new"], beta * m + g, atol=1e-15)


def test_decode_identities_order_three():
    rng = np.random.default_rng(6)
    shape, chunk, k = (8, 6, 10), (4, 3, 5), 11
    lr, wd = 1e-2, 0.1
    x = rng.standard_normal(shape)
    W = 3
    outs = [ond.compress_tensor(rng.standard_normal(shape), rng.standard_normal(shape), chunk, k, 0.9) for _ in range(W)]
    pay = [o["records"] for o in outs]
    # linearity in the workers: R = sum_w IDCT(records_w), rebuilt with scipy from the fp32 record values
    want = np.zeros(shape)
    M = int(np.prod(chunk))
    for o in outs:
        dense = np.zeros((o["records"].shape[0], M))
        for c in range(dense.shape[0]):
            dense[c, o["records"]["idx"][c]] = o["records"]["val"][c].astype(np.float64)
        grid = tuple(n // s for n, s in zip(shape, chunk))
        per = np.stack([scipy.fft.idctn(d.reshape(chunk), norm="ortho") for d in dense]).reshape(grid + chunk)
        want += ond.unblocks(per, shape)
    dec = ond.decode_tensor(pay, x, chunk, lr, wd)
    np.testing.assert_allclose(dec["R"], want, atol=1e-12)
    np.testing.assert_allclose(dec["x_new"], x - lr * (np.sign(want) + wd * x), atol=1e-15)
    # mean: same signs, R / W; identity update is linear in R
    mean = ond.decode_tensor(pay, x, chunk, lr, wd, agg=ond.AGG_MEAN, phi=ond.PHI_IDENTITY)
    np.testing.assert_allclose(mean["R"], want / W, atol=1e-12)
    np.testing.assert_allclose(mean["x_new"], x - lr * (want / W + wd * x), atol=1e-15)
    # all-zero record values: x_new = x (1 - lr wd) exactly
    zero = [p.copy() for p in pay]
    for p in zero:
        p["val"] = 0.0
    np.testing.assert_array_equal(ond.decode_tensor(zero, x, chunk, lr, wd)["x_new"], x - lr * (0.0 + wd * x))
    # W = 1 with k = M: decode rebuilds beta m + g, so the update is its sign
    g1, m1 = rng.standard_normal(shape), rng.standard_normal(shape)
    one = ond.compress_tensor(g1, m1, chunk, M, 0.9)
    d1 = ond.decode_tensor([one["records"]], x, chunk, lr, wd)
    np.testing.assert_allclose(d1["R"], 0.9 * m1 + g1, atol=1e-6)  # record values are fp32
    # count-normalised mean by hand on one chunk
    rec = np.zeros((3, 1, 2), dtype=ond.RECORD_DTYPE)
    rec["idx"] = [[[0, 5]], [[0, 7]], [[5, 9]]]
    rec["val"] = [[[1.0, 2.0]], [[3.0, 4.0]], [[6.0, 8.0]]]
    S = np.zeros(60)
    S[[0, 5, 7, 9]] = [(1 + 3) / 2, (2 + 6) / 2, 4.0, 8.0]
    got = ond.decode_chunks(rec, np.zeros((1, 60)), chunk, 1.0, 0.0, agg=ond.AGG_COUNT_MEAN, phi=ond.PHI_IDENTITY)
    np.testing.assert_allclose(got["R"][0], scipy.fft.idctn(S.reshape(chunk), norm="ortho").reshape(-1), atol=1e-13)


def test_forced_index_continuation():
    rng = np.random.default_rng(7)
    chunk = (4, 6)
    g, m = rng.standard_normal((5, 24)), rng.standard_normal((5, 24))
    free = ond.compress_chunks(g, m, chunk, 5, 0.9)
    forced = ond.compress_chunks(g, m, chunk, 5, 0.9, forced_idx=free["idx"])
    np.testing.assert_array_equal(forced["m_new"], free["m_new"])
    other = np.tile(np.arange(5, dtype=np.int32), (5, 1))
    f2 = ond.compress_chunks(g, m, chunk, 5, 0.9, forced_idx=other)
    for c in range(5):
        Q = scipy.fft.dctn((0.9 * m[c] + g[c]).reshape(chunk), norm="ortho").reshape(-1)
        Q[:5] = 0.0
        np.testing.assert_allclose(f2["m_new"][c], scipy.fft.idctn(Q.reshape(chunk), norm="ortho").reshape(-1), atol=1e-12)
