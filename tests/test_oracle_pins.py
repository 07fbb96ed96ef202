"""Pins for the fp64 CPU oracle: it is checked against what the paper and the mathematics fix,
never against itself.  Each group names the passage of the paper that fixes the property.
A plausible mistake (dropped term, wrong sign or index, transposed operand) fails one of them.
"""
import itertools
import math
import os

import numpy as np
import pytest
import scipy.fft

from oracle import demo_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
SIZES = [1, 2, 4, 8, 32, 64, 128]


def _read_table(name):
    rows = []
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                rows.append(line.split())
    return rows


# --------------------------------------------------------------------------------------------
# DCT basis: orthonormal DCT-II ("unitary", P^T = P^-1; appendix B.1.2; Section 2.1)
# --------------------------------------------------------------------------------------------
def test_dct_matrix_textbook_values():
    for s, u, n, v in _read_table("dct_textbook_values.txt"):
        C = orc.dct_matrix(int(s))
        assert abs(C[int(u), int(n)] - float(v)) < 1e-12


@pytest.mark.parametrize("s", SIZES)
def test_dct_matrix_is_unitary(s):
    C = orc.dct_matrix(s)
    assert np.max(np.abs(C @ C.T - np.eye(s))) <= 1e-12
    assert np.max(np.abs(C.T @ C - np.eye(s))) <= 1e-12


@pytest.mark.parametrize("s", SIZES)
def test_dct_matrix_structure(s):
    C = orc.dct_matrix(s)
    # row 0 is the constant 1/sqrt(s); every other row sums to zero
    assert np.allclose(C[0], 1.0 / math.sqrt(s), atol=1e-15)
    if s > 1:
        assert np.max(np.abs(C[1:].sum(axis=1))) < 1e-12
    # mirror symmetry C[u][s-1-n] = (-1)^u C[u][n]
    signs = (-1.0) ** np.arange(s)
    assert np.max(np.abs(C[:, ::-1] - signs[:, None] * C)) < 1e-13


@pytest.mark.parametrize("s", SIZES)
def test_dct_matrix_matches_library_dct(s):
    # a library routine the closed form must reduce to: column n of C is the DCT-II of e_n
    C = orc.dct_matrix(s)
    ref = scipy.fft.dct(np.eye(s), type=2, norm="ortho", axis=0)
    assert np.max(np.abs(C - ref)) < 1e-13


# --------------------------------------------------------------------------------------------
# Separable transform T: d=2 is P0 B P1^T (Section 2.1), explicit index formula (appendix B.1.2)
# --------------------------------------------------------------------------------------------
def test_forward_brute_force_8x8_from_index_formula():
    rng = np.random.default_rng(7)
    s = 8
    B = rng.standard_normal((s, s))
    Q = orc.forward(B)
    pi = math.pi
    for u, v in itertools.product(range(s), range(s)):
        acc = 0.0
        for i, j in itertools.product(range(s), range(s)):
            au = math.sqrt(1 / s) if u == 0 else math.sqrt(2 / s)
            av = math.sqrt(1 / s) if v == 0 else math.sqrt(2 / s)
            acc += (au * math.cos(pi * (2 * i + 1) * u / (2 * s))) * (av * math.cos(pi * (2 * j + 1) * v / (2 * s))) * B[i, j]
        assert abs(Q[u, v] - acc) < 1e-12


@pytest.mark.parametrize("s", [8, 32, 64, 128])
def test_forward_and_inverse_match_library_2d(s):
    rng = np.random.default_rng(s)
    B = rng.standard_normal((s, s)) * np.exp(rng.standard_normal((s, 1)))  # not symmetric
    Q = orc.forward(B)
    assert np.max(np.abs(Q - scipy.fft.dctn(B, type=2, norm="ortho"))) < 1e-11
    R = orc.inverse(Q)
    assert np.max(np.abs(R - B)) < 1e-11
    assert np.max(np.abs(orc.inverse(B) - scipy.fft.idctn(B, type=2, norm="ortho"))) < 1e-11


@pytest.mark.parametrize("s", [8, 32, 64, 128])
def test_forward_and_inverse_match_library_1d(s):
    rng = np.random.default_rng(100 + s)
    b = rng.standard_normal(s)
    q = orc.forward(b)
    assert np.max(np.abs(q - scipy.fft.dct(b, type=2, norm="ortho"))) < 1e-12
    assert np.max(np.abs(orc.inverse(q) - b)) < 1e-12


def test_forward_via_fft_of_padded_signal():
    # DCT-II from an FFT of the zero-padded length-2s signal, phase-rotated and scaled
    s = 64
    rng = np.random.default_rng(3)
    b = rng.standard_normal(s)
    F = np.fft.fft(np.concatenate([b, np.zeros(s)]))[:s]
    X = np.real(F * np.exp(-1j * np.pi * np.arange(s) / (2 * s)))
    X *= np.sqrt(2.0 / s)
    X[0] /= np.sqrt(2.0)
    assert np.max(np.abs(orc.forward(b) - X)) < 1e-12


@pytest.mark.parametrize("s", [8, 64])
def test_parseval_constant_and_basis_tiles(s):
    rng = np.random.default_rng(11)
    B = rng.standard_normal((s, s))
    Q = orc.forward(B)
    assert abs(np.sum(B * B) - np.sum(Q * Q)) <= 1e-12 * np.sum(B * B)
    # constant tile a -> single DC coefficient a*s (1-D: a*sqrt(s))
    Qc = orc.forward(np.full((s, s), 0.37))
    assert abs(Qc[0, 0] - 0.37 * s) < 1e-12
    Qc[0, 0] = 0.0
    assert np.max(np.abs(Qc)) < 1e-12
    qc = orc.forward(np.full(s, 0.37))
    assert abs(qc[0] - 0.37 * math.sqrt(s)) < 1e-12
    # tile = outer(C[u0], C[v0]) -> a single 1 at (u0, v0): catches a transposed operand
    C = orc.dct_matrix(s)
    u0, v0 = 2, 5
    Qb = orc.forward(np.outer(C[u0], C[v0]))
    E = np.zeros((s, s))
    E[u0, v0] = 1.0
    assert np.max(np.abs(Qb - E)) < 1e-12
    # linearity
    B2 = rng.standard_normal((s, s))
    assert np.max(np.abs(orc.forward(2.0 * B - 3.0 * B2) - (2.0 * Q - 3.0 * orc.forward(B2)))) < 1e-11


# --------------------------------------------------------------------------------------------
# Blocking operator: the paper's worked 128 x 512 / 16 x 32 example (appendix B.1.2)
# --------------------------------------------------------------------------------------------
def test_blocking_paper_example():
    kv = {k: int(v) for k, v in _read_table("paper_compression_ratios.txt")}
    n0, n1, s0, s1 = kv["block_example_n0"], kv["block_example_n1"], kv["block_example_s0"], kv["block_example_s1"]
    assert (n0 // s0, n1 // s1) == (kv["block_example_c0"], kv["block_example_c1"])
    X = np.arange(n0 * n1, dtype=np.float64).reshape(n0, n1)  # index-valued matrix
    for k0, k1 in [(0, 0), (7, 15), (3, 9)]:
        B = orc.block_extract(X, s0, s1, k0, k1)
        assert B.shape == (s0, s1)
        for j0, j1 in [(0, 0), (15, 31), (4, 17)]:
            assert B[j0, j1] == (s0 * k0 + j0) * n1 + (s1 * k1 + j1)
    B00 = orc.block_extract(X, s0, s1, 0, 0)
    assert B00[0, 31] == 31 and B00[15, 0] == 15 * n1 and B00[1, 1] == n1 + 1


# --------------------------------------------------------------------------------------------
# Top-k: k largest magnitudes, ||Q_hat||_0 = k (Section 2.1); thr = k-th largest (appendix alg.)
# --------------------------------------------------------------------------------------------
@pytest.mark.parametrize("M,k", [(64, 4), (64, 64), (4096, 32), (4096, 1), (64, 128)])
def test_topk_equals_full_sort(M, k):
    rng = np.random.default_rng(M + k)
    q = rng.standard_normal(M)
    idx, a_k, a_k1 = orc.topk(q, k)
    k_eff = min(k, M)
    order = np.lexsort((np.arange(M), -np.abs(q)))  # primary: -|q|, secondary: index
    assert np.array_equal(idx, np.sort(order[:k_eff]).astype(np.int32))
    assert len(set(idx.tolist())) == k_eff and np.all(np.diff(idx) > 0)
    assert a_k == np.abs(q)[order[k_eff - 1]]
    assert a_k1 == (np.abs(q)[order[k_eff]] if k_eff < M else 0.0)
    sel = np.zeros(M, bool)
    sel[idx] = True
    if k_eff < M:
        assert np.abs(q)[sel].min() >= a_k >= np.abs(q)[~sel].max()


def test_topk_brute_force_tiny():
    # every subset of size k of an 8-vector: the chosen set maximises the kept energy
    rng = np.random.default_rng(5)
    q = rng.standard_normal(8)
    idx, _, _ = orc.topk(q, 3)
    best = max(itertools.combinations(range(8), 3), key=lambda c: sum(q[i] ** 2 for i in c))
    assert sorted(best) == idx.tolist()


def test_topk_ties_go_to_lowest_index():
    q = np.array([1.0, -2.0, 2.0, 0.5, 2.0, -2.0, 0.1, 2.0])
    idx, a_k, a_k1 = orc.topk(q, 3)
    assert idx.tolist() == [1, 2, 4] and a_k == 2.0 and a_k1 == 2.0
    idx, _, _ = orc.topk(np.zeros(16), 4)
    assert idx.tolist() == [0, 1, 2, 3]


# --------------------------------------------------------------------------------------------
# CompressChunks: residual identities; sqrt(1-k/M) bound with its equality case (appendix lemma
# on the top-k error and the isometric-transform remark); lossless k = M
# --------------------------------------------------------------------------------------------
@pytest.mark.parametrize("s,rows,k", [(8, 8, 4), (8, 1, 4), (64, 64, 32), (64, 1, 32), (32, 32, 8)])
def test_compress_chunk_identities(s, rows, k):
    rng = np.random.default_rng(s * 1000 + rows + k)
    M = rows * s
    n = 3
    g = rng.standard_normal((n, M)) * 0.01
    m = rng.standard_normal((n, M)) * 0.1
    beta = 0.999
    out = orc.compress_chunks(g, m, s, rows, k, beta)
    shape = (s, s) if rows == s else (s,)
    for c in range(n):
        B = (beta * m[c] + g[c]).reshape(shape)
        Qlib = (scipy.fft.dctn(B, type=2, norm="ortho") if rows == s else scipy.fft.dct(B, type=2, norm="ortho")).reshape(-1)
        assert np.max(np.abs(out["Q"][c] - Qlib)) < 1e-12  # m <- beta*m + g, then DCT
        idx = out["idx"][c]
        assert np.array_equal(idx, orc.topk(Qlib, k)[0])
        assert np.max(np.abs(out["val"][c] - Qlib[idx])) < 1e-12
        mn = out["m_new"][c].reshape(shape)
        Qres = orc.forward(mn).reshape(-1)
        mask = np.zeros(M, bool)
        mask[idx] = True
        assert np.max(np.abs(Qres[mask])) < 1e-12  # removed exactly the transmitted part
        assert np.max(np.abs(Qres[~mask] - Qlib[~mask])) < 1e-12
        # energy identity and reconstruction identity
        assert abs(np.sum(mn**2) - (np.sum(Qlib**2) - np.sum(Qlib[idx] ** 2))) < 1e-12
        Qsp = np.zeros(M)
        Qsp[idx] = out["val"][c]
        assert np.max(np.abs(orc.inverse(Qsp.reshape(shape)) + mn - B)) < 1e-12
        # error bound of the top-k lemma under an isometry
        k_eff = min(k, M)
        assert np.linalg.norm(mn) <= math.sqrt(1 - k_eff / M) * np.linalg.norm(B) + 1e-12


def test_residual_bound_equality_case():
    s, k = 8, 4
    rng = np.random.default_rng(2)
    a = 0.3
    Qeq = a * rng.choice([-1.0, 1.0], size=(s, s))  # all coefficient magnitudes equal
    B = orc.inverse(Qeq)
    out = orc.compress_chunks(B.reshape(1, -1), np.zeros((1, s * s)), s, s, k, 0.5)
    lhs = np.linalg.norm(out["m_new"][0])
    rhs = math.sqrt(1 - k / (s * s)) * np.linalg.norm(B)
    assert abs(lhs - rhs) < 1e-12


@pytest.mark.parametrize("s,rows", [(8, 8), (8, 1), (32, 32)])
def test_lossless_when_k_equals_M(s, rows):
    rng = np.random.default_rng(9)
    M = rows * s
    W = 3
    beta, lr, wd = 0.9, 1e-3, 0.1
    g = rng.standard_normal((W, 2, M))
    m = rng.standard_normal((W, 2, M))
    recs = np.zeros((W, 2, M), dtype=orc.RECORD_DTYPE)
    total = np.zeros((2, M))
    for w in range(W):
        out = orc.compress_chunks(g[w], m[w], s, rows, M, beta)
        B = beta * m[w] + g[w]
        assert np.max(np.abs(out["m_new"])) <= 1e-12 * np.max(np.abs(B))  # zero residual
        recs[w]["idx"] = out["idx"]
        recs[w]["val"] = out["val"].astype(np.float32)
        total += B
    x = rng.standard_normal((2, M)) * 0.02
    dec = orc.decode_chunks(recs, x, s, rows, lr, wd)
    big = np.abs(total) > 1e-5  # away from rounding of the fp32 payload values
    assert np.array_equal(np.sign(dec["R"])[big], np.sign(total)[big])  # update = sign(sum_w m_w)
    assert np.max(np.abs(dec["x_new"] - (x - lr * (np.sign(dec["R"]) + wd * x)))) < 1e-15


# --------------------------------------------------------------------------------------------
# Decompress&Aggregate + update (Algorithm 1 server side; update x - eta (sgn + lambda x))
# --------------------------------------------------------------------------------------------
def test_decode_single_worker_reconstructs_removed_part():
    s, rows, k = 8, 8, 5
    rng = np.random.default_rng(4)
    M = s * s
    g = rng.standard_normal((4, M))
    m = rng.standard_normal((4, M))
    beta = 0.999
    out = orc.compress_chunks(g, m, s, rows, k, beta)
    recs = np.zeros((1, 4, k), dtype=orc.RECORD_DTYPE)
    recs[0]["idx"] = out["idx"]
    recs[0]["val"] = out["val"].astype(np.float32)
    dec = orc.decode_chunks(recs, np.zeros((4, M)), s, rows, 1e-3, 0.0)
    assert np.max(np.abs(dec["R"] - ((beta * m + g) - out["m_new"]))) < 1e-6  # fp32 payload rounding


def test_decode_zero_payload_and_sign_zero():
    s, rows, k, W = 8, 8, 4, 2
    M = s * s
    recs = np.zeros((W, 3, k), dtype=orc.RECORD_DTYPE)
    recs["idx"] = np.arange(k, dtype=np.int32)
    x = np.random.default_rng(1).standard_normal((3, M))
    lr, wd = 1e-3, 0.1
    dec = orc.decode_chunks(recs, x, s, rows, lr, wd)
    assert np.all(dec["R"] == 0.0)
    assert np.max(np.abs(dec["x_new"] - x * (1 - lr * wd))) < 1e-15  # sign(0) = 0


def test_decode_linearity_collisions_and_step_size():
    s, rows, k, W = 8, 8, 6, 4
    M = s * s
    rng = np.random.default_rng(8)
    recs = np.zeros((W, 2, k), dtype=orc.RECORD_DTYPE)
    for w in range(W):
        for c in range(2):
            recs[w, c]["idx"] = np.sort(rng.choice(16, size=k, replace=False))  # small range -> collisions
            recs[w, c]["val"] = rng.standard_normal(k).astype(np.float32)
    x = rng.standard_normal((2, M))
    lr = 2e-3
    dec = orc.decode_chunks(recs, x, s, rows, lr, 0.0)
    Rsum = np.zeros((2, M))
    for w in range(W):
        for c in range(2):
            S = np.zeros(M)
            S[recs[w, c]["idx"]] = recs[w, c]["val"].astype(np.float64)
            Rsum[c] += scipy.fft.idctn(S.reshape(s, s), type=2, norm="ortho").reshape(-1)
    assert np.max(np.abs(dec["R"] - Rsum)) < 1e-12
    # weight decay 0: every parameter moves by exactly 0 or +-lr
    step = dec["x_new"] - x
    assert np.all(np.isclose(np.abs(step), lr, rtol=0, atol=1e-15) | (step == 0.0))
    assert np.array_equal(np.sign(-step), np.sign(Rsum))


def test_decode_degenerates_to_signum_at_chunk_size_one():
    # s = 1, k = 1: C = [[1]], nothing is dropped, update is the sign of the summed momentum
    rng = np.random.default_rng(12)
    W, n = 3, 10
    g = rng.standard_normal((W, n, 1))
    m = rng.standard_normal((W, n, 1))
    recs = np.zeros((W, n, 1), dtype=orc.RECORD_DTYPE)
    for w in range(W):
        out = orc.compress_chunks(g[w], m[w], 1, 1, 1, 0.9)
        assert np.all(out["m_new"] == 0.0)
        recs[w]["idx"] = out["idx"]
        recs[w]["val"] = out["val"].astype(np.float32)
    x = rng.standard_normal((n, 1))
    dec = orc.decode_chunks(recs, x, 1, 1, 1e-2, 0.0)
    assert np.array_equal(np.sign(x - dec["x_new"]).reshape(-1), np.sign((0.9 * m + g).sum(axis=0)).reshape(-1))


# --------------------------------------------------------------------------------------------
# Whole-tensor drivers: chunk order is row-major over the chunk grid; 1-D tensors use length-s
# segments with the same k (k_eff = min(k, s))
# --------------------------------------------------------------------------------------------
def test_tensor_driver_matches_chunk_routine_and_chunk_order():
    s, k, beta = 8, 4, 0.999
    rng = np.random.default_rng(21)
    n0, n1 = 24, 40
    g = rng.standard_normal((n0, n1)) * 0.01
    m = rng.standard_normal((n0, n1)) * 0.1
    out = orc.compress_tensor(g, m, s, k, beta)
    c1 = n1 // s
    for k0, k1 in [(0, 0), (2, 4), (1, 3)]:
        gt = g[k0 * s:(k0 + 1) * s, k1 * s:(k1 + 1) * s].reshape(1, -1)
        mt = m[k0 * s:(k0 + 1) * s, k1 * s:(k1 + 1) * s].reshape(1, -1)
        ch = orc.compress_chunks(gt, mt, s, s, k, beta)
        c = k0 * c1 + k1
        assert np.array_equal(out["records"][c]["idx"], ch["idx"][0])
        assert np.array_equal(out["records"][c]["val"], ch["val"][0].astype(np.float32))
        assert np.array_equal(out["m_new"][k0 * s:(k0 + 1) * s, k1 * s:(k1 + 1) * s].reshape(-1), ch["m_new"][0])
    # decode driver against the chunk routine
    x = rng.standard_normal((n0, n1)) * 0.02
    dec = orc.decode_tensor([out["records"], out["records"]], x, s, k, 1e-3, 0.1)
    c = 1 * c1 + 3
    recs = np.stack([out["records"][c:c + 1], out["records"][c:c + 1]])
    dch = orc.decode_chunks(recs, x[s:2 * s, 3 * s:4 * s].reshape(1, -1), s, s, 1e-3, 0.1)
    assert np.array_equal(dec["x_new"][s:2 * s, 3 * s:4 * s].reshape(-1), dch["x_new"][0])


def test_tensor_driver_1d_and_shape_errors():
    s, k = 8, 16  # k > s: lossless on a 1-D segment
    rng = np.random.default_rng(22)
    g = rng.standard_normal(64)
    m = rng.standard_normal(64)
    out = orc.compress_tensor(g, m, s, k, 0.5)
    assert out["records"].shape == (8, 8)
    assert np.max(np.abs(out["m_new"])) < 1e-12
    q = scipy.fft.dct((0.5 * m + g)[8:16], type=2, norm="ortho")
    assert np.max(np.abs(out["val64"][1] - q)) < 1e-12
    with pytest.raises(ValueError):
        orc.compress_tensor(np.zeros(60), np.zeros(60), s, k, 0.5)
    with pytest.raises(ValueError):
        orc.compress_tensor(np.zeros((12, 16)), np.zeros((12, 16)), s, k, 0.5)


def test_payload_volume_matches_paper_ratios():
    kv = {k: int(v) for k, v in _read_table("paper_compression_ratios.txt")}
    s, k, W = kv["s"], kv["k"], kv["workers"]
    n0 = n1 = 2 * s
    out = orc.compress_tensor(np.ones((n0, n1)), np.zeros((n0, n1)), s, k, 0.9)
    n_records = out["records"].size
    assert n_records == (n0 // s) * (n1 // s) * k
    assert (n0 * n1) // n_records == kv["tx_reduction"]  # coefficients sent: M / k
    assert (n0 * n1) // (W * n_records) == kv["rx_reduction"]  # received from 8 workers


# --------------------------------------------------------------------------------------------
# alpha-scaled momentum subtraction (Section 2.1 "Momentum Subtraction as Error Feedback")
# --------------------------------------------------------------------------------------------
def test_alpha_scaled_momentum_subtraction():
    s, rows, k, beta = 8, 8, 6, 0.999
    rng = np.random.default_rng(31)
    g = rng.standard_normal((3, 64)) * 0.01
    m = rng.standard_normal((3, 64)) * 0.1
    B = beta * m + g
    full = orc.compress_chunks(g, m, s, rows, k, beta)  # default alpha = 1
    one = orc.compress_chunks(g, m, s, rows, k, beta, alpha=1.0)
    assert np.array_equal(full["m_new"], one["m_new"])
    zero = orc.compress_chunks(g, m, s, rows, k, beta, alpha=0.0)
    assert np.array_equal(zero["m_new"], B)  # nothing removed
    assert np.array_equal(zero["idx"], full["idx"]) and np.array_equal(zero["val"], full["val"])  # payload unaffected
    a = 0.2
    part = orc.compress_chunks(g, m, s, rows, k, beta, alpha=a)
    # linear in alpha: B - alpha * IDCT(kept), with IDCT(kept) = B - m_new(alpha = 1)
    assert np.max(np.abs(part["m_new"] - (B - a * (B - full["m_new"])))) < 1e-14
    # the transmitted part is removed only partially: DCT of the residual keeps (1 - alpha) of the kept coefficients
    for c in range(3):
        Qres = orc.forward(part["m_new"][c].reshape(s, s)).reshape(-1)
        assert np.max(np.abs(Qres[full["idx"][c]] - (1 - a) * full["val"][c])) < 1e-12
    t = orc.compress_tensor(g.reshape(24, 8), m.reshape(24, 8), s, k, beta, alpha=a)
    assert np.max(np.abs(t["m_new"].reshape(3, 64) - part["m_new"])) < 1e-14


# --------------------------------------------------------------------------------------------
# Aggregation variants and phi = identity (Section 2.1: AvgAllGather, phi; appendix algorithm
# "Sparse Top-k Averaging": sum / per-coordinate count, 0/0 = 0)
# --------------------------------------------------------------------------------------------
def _recs(W, n, k, idx_lists, val_lists):
    r = np.zeros((W, n, k), dtype=orc.RECORD_DTYPE)
    for w in range(W):
        r[w, 0]["idx"] = idx_lists[w]
        r[w, 0]["val"] = np.asarray(val_lists[w], dtype=np.float32)
    return r


def test_aggregation_variants_hand_example():
    s, rows, M = 4, 1, 4  # 1-D segments of 4: coefficients are easy to follow by hand
    # three workers; coordinate 0 sent by all, 1 by two, 2 by one, 3 by none
    recs = _recs(3, 1, 2, [[0, 1], [0, 1], [0, 2]], [[3.0, 1.0], [6.0, -2.0], [-3.0, 8.0]])
    x = np.zeros((1, M))
    want_sum = np.array([6.0, -1.0, 8.0, 0.0])
    want_mean = want_sum / 3.0
    want_cnt = np.array([6.0 / 3, -1.0 / 2, 8.0 / 1, 0.0])  # 0/0 = 0 at coordinate 3
    for agg, want in [(orc.AGG_SUM, want_sum), (orc.AGG_MEAN, want_mean), (orc.AGG_COUNT_MEAN, want_cnt)]:
        out = orc.decode_chunks(recs, x, s, rows, 1.0, 0.0, agg=agg, phi=orc.PHI_IDENTITY)
        R = scipy.fft.idct(want, type=2, norm="ortho")
        assert np.max(np.abs(out["R"][0] - R)) < 1e-14
        assert np.max(np.abs(out["x_new"][0] - (x[0] - R))) < 1e-14  # phi = identity, lr = 1, wd = 0


def test_count_mean_limits_and_identity_update():
    s, rows, k, W = 8, 8, 5, 4
    M = s * s
    rng = np.random.default_rng(41)
    x = rng.standard_normal((2, M)) * 0.02
    # disjoint index sets: count-normalised == sum; identical index sets: count-normalised == mean
    dis = np.zeros((W, 2, k), dtype=orc.RECORD_DTYPE)
    same = np.zeros((W, 2, k), dtype=orc.RECORD_DTYPE)
    for w in range(W):
        for c in range(2):
            dis[w, c]["idx"] = np.arange(w * k, (w + 1) * k)
            same[w, c]["idx"] = np.arange(3, 3 + k)
            dis[w, c]["val"] = rng.standard_normal(k).astype(np.float32)
            same[w, c]["val"] = rng.standard_normal(k).astype(np.float32)
    a = orc.decode_chunks(dis, x, s, rows, 1e-3, 0.1, agg=orc.AGG_COUNT_MEAN)
    b = orc.decode_chunks(dis, x, s, rows, 1e-3, 0.1, agg=orc.AGG_SUM)
    assert np.array_equal(a["R"], b["R"]) and np.array_equal(a["x_new"], b["x_new"])
    a = orc.decode_chunks(same, x, s, rows, 1e-3, 0.1, agg=orc.AGG_COUNT_MEAN, phi=orc.PHI_IDENTITY)
    b = orc.decode_chunks(same, x, s, rows, 1e-3, 0.1, agg=orc.AGG_MEAN, phi=orc.PHI_IDENTITY)
    assert np.max(np.abs(a["R"] - b["R"])) < 1e-15
    # the mean has the sign of the sum; identity applies R itself: x - lr (R + wd x)
    c = orc.decode_chunks(same, x, s, rows, 1e-3, 0.1, agg=orc.AGG_SUM)
    d = orc.decode_chunks(same, x, s, rows, 1e-3, 0.1, agg=orc.AGG_MEAN)
    assert np.array_equal(c["x_new"], d["x_new"])
    assert np.max(np.abs(b["x_new"] - (x - 1e-3 * (b["R"] + 0.1 * x)))) < 1e-16
    assert np.max(np.abs(b["R"] - c["R"] / W)) < 1e-15


# --------------------------------------------------------------------------------------------
# Other orthonormal bases (Section 4.2, "Choice of Linear Projections"): identity, and a Gaussian
# matrix orthonormalised by the Gram-Schmidt process
# --------------------------------------------------------------------------------------------
def test_gram_schmidt_hand_example_and_library_qr():
    # 2 x 2 by hand: rows (3,4), (1,0) -> (0.6,0.8), then (1,0) - 0.6*(0.6,0.8) = (0.64,-0.48) -> (0.8,-0.6)
    P = orc.gram_schmidt(np.array([[3.0, 4.0], [1.0, 0.0]]))
    assert np.max(np.abs(P - np.array([[0.6, 0.8], [0.8, -0.6]]))) < 1e-15
    rng = np.random.default_rng(5)
    for s in (8, 32, 64, 128):
        G = rng.standard_normal((s, s))
        P = orc.gram_schmidt(G)
        assert np.max(np.abs(P @ P.T - np.eye(s))) < 1e-12
        # rows orthonormalised in order: G = L P with L lower triangular, positive diagonal
        L = G @ P.T
        assert np.max(np.abs(np.triu(L, 1))) < 1e-11 and np.all(np.diag(L) > 0)
        assert np.max(np.abs(P[0] - G[0] / np.linalg.norm(G[0]))) < 1e-15
        # the library's QR of G^T gives the same vectors once its signs are fixed
        Qm, Rm = np.linalg.qr(G.T)
        assert np.max(np.abs(P - (Qm * np.sign(np.diag(Rm))).T)) < 1e-10
    with pytest.raises(ValueError):
        orc.gram_schmidt(np.ones((4, 4)))


def test_identity_basis_is_plain_topk_of_the_momentum():
    s, rows, k, n = 8, 8, 5, 6
    M = s * s
    rng = np.random.default_rng(6)
    g, m = rng.standard_normal((n, M)), rng.standard_normal((n, M))
    out = orc.compress_chunks(g, m, s, rows, k, 0.9, basis=np.eye(s))
    B = 0.9 * m + g
    for c in range(n):
        want = np.sort(np.argsort(-np.abs(B[c]), kind="stable")[:k])
        assert np.array_equal(out["idx"][c], want)
        assert np.array_equal(out["val"][c], B[c][want]) and np.array_equal(out["Q"][c], B[c])
        keep = B[c].copy()
        keep[want] = 0.0
        assert np.array_equal(out["m_new"][c], keep)
    # decode with the identity: the scattered sum itself drives the update
    recs = np.zeros((2, n, k), dtype=orc.RECORD_DTYPE)
    recs[0]["idx"], recs[0]["val"] = out["idx"], out["val"].astype(np.float32)
    recs[1]["idx"], recs[1]["val"] = out["idx"], (2.0 * out["val"]).astype(np.float32)
    x = rng.standard_normal((n, M)) * 0.02
    dec = orc.decode_chunks(recs, x, s, rows, 1e-3, 0.1, basis=np.eye(s))
    S = np.zeros((n, M))
    for c in range(n):
        S[c][out["idx"][c]] = recs[0][c]["val"].astype(np.float64) + recs[1][c]["val"].astype(np.float64)
    assert np.array_equal(dec["R"], S)
    assert np.max(np.abs(dec["x_new"] - (x - 1e-3 * (np.sign(S) + 0.1 * x)))) < 1e-17


@pytest.mark.parametrize("s,rows", [(8, 8), (32, 32), (64, 1)])
def test_random_orthonormal_basis_identities(s, rows):
    M, k, n = s * rows, 7, 3
    rng = np.random.default_rng(7)
    P = orc.gram_schmidt(rng.standard_normal((s, s)))
    g, m = rng.standard_normal((n, M)), rng.standard_normal((n, M))
    out = orc.compress_chunks(g, m, s, rows, k, 0.999, basis=P)
    B = 0.999 * m + g
    for c in range(n):
        # rows of P are the basis vectors: Q = P B P^T (2-D), q = P b (1-D); P is not symmetric, so
        # a transposed operand fails here
        Qw = P @ B[c].reshape(rows, s) @ P.T if rows > 1 else P @ B[c]
        assert np.max(np.abs(out["Q"][c] - Qw.reshape(-1))) < 1e-12
        assert abs(np.sum(out["Q"][c] ** 2) - np.sum(B[c] ** 2)) < 1e-10 * np.sum(B[c] ** 2)
        Qs = np.zeros(M)
        Qs[out["idx"][c]] = out["val"][c]
        back = P.T @ Qs.reshape(rows, s) @ P if rows > 1 else P.T @ Qs
        assert np.max(np.abs(back.reshape(-1) + out["m_new"][c] - B[c])) < 1e-12
    # W = 1 decode rebuilds what compress removed
    recs = np.zeros((1, n, k), dtype=orc.RECORD_DTYPE)
    recs[0]["idx"], recs[0]["val"] = out["idx"], out["val"].astype(np.float32)
    dec = orc.decode_chunks(recs, np.zeros((n, M)), s, rows, 1.0, 0.0, basis=P, phi=orc.PHI_IDENTITY)
    assert np.max(np.abs(dec["R"] - (B - out["m_new"]))) < 1e-6


def test_explicit_dct_basis_equals_default_and_tensor_driver_takes_a_basis():
    s, k = 8, 4
    rng = np.random.default_rng(8)
    g, m = rng.standard_normal((16, 24)), rng.standard_normal((16, 24))
    a = orc.compress_tensor(g, m, s, k, 0.9)
    b = orc.compress_tensor(g, m, s, k, 0.9, basis=orc.dct_matrix(s))
    assert np.array_equal(a["records"], b["records"]) and np.array_equal(a["m_new"], b["m_new"])
    P = orc.gram_schmidt(rng.standard_normal((s, s)))
    t = orc.compress_tensor(g, m, s, k, 0.9, basis=P)
    # chunk (1, 2) of the tensor driver == the chunk routine on that tile
    tile = lambda X: orc.block_extract(X, s, s, 1, 2).reshape(1, -1)
    c = orc.compress_chunks(tile(g), tile(m), s, s, k, 0.9, basis=P)
    assert np.array_equal(t["records"][1 * 3 + 2]["idx"], c["idx"][0])
    assert np.array_equal(orc.block_extract(t["m_new"], s, s, 1, 2).reshape(-1), c["m_new"][0])
    x = rng.standard_normal((16, 24)) * 0.02
    d1 = orc.decode_tensor([a["records"]], x, s, k, 1e-3, 0.1)
    d2 = orc.decode_tensor([a["records"]], x, s, k, 1e-3, 0.1, basis=orc.dct_matrix(s))
    assert np.array_equal(d1["x_new"], d2["x_new"])
    d3 = orc.decode_tensor([t["records"]], x, s, k, 1e-3, 0.1, basis=P)
    R = orc.block_extract(d3["R"], s, s, 1, 2)
    Qs = np.zeros(s * s)
    Qs[c["idx"][0]] = c["val"][0].astype(np.float32)
    assert np.max(np.abs(R - P.T @ Qs.reshape(s, s) @ P)) < 1e-12


# --------------------------------------------------------------------------------------------
# Forced-index continuation of the C oracle (the comparison harness uses it where several top-k
# sets are valid): with a given index set the residual is B - alpha * IDCT(Q restricted to the set)
# (Section 2.1 "Momentum Subtraction as Error Feedback"), whatever the magnitudes say.
# --------------------------------------------------------------------------------------------
def _forced_case(seed, n, s, rows, k):
    rng = np.random.default_rng(seed)
    M = rows * s
    g = rng.standard_normal((n, M))
    m = rng.standard_normal((n, M))
    return g, m, M, min(k, M)


@pytest.mark.parametrize("s,rows,k", [(8, 8, 5), (16, 16, 7), (8, 1, 3)])
def test_forced_index_with_the_oracles_own_set_changes_nothing(s, rows, k):
    g, m, M, k_eff = _forced_case(11, 5, s, rows, k)
    beta = 0.9
    free = orc.compress_chunks(g, m, s, rows, k, beta)
    forced = orc.compress_chunks(g, m, s, rows, k, beta, forced_idx=free["idx"])
    assert np.array_equal(forced["idx"], free["idx"])
    assert np.array_equal(forced["val"], free["val"])
    assert np.array_equal(forced["m_new"], free["m_new"])  # bit for bit
    assert np.array_equal(forced["Q"], free["Q"])


@pytest.mark.parametrize("alpha", [1.0, 0.25])
def test_forced_index_with_another_set_follows_the_definition(alpha):
    s, rows, k, beta = 8, 8, 6, 0.75
    g, m, M, k_eff = _forced_case(12, 4, s, rows, k)
    rng = np.random.default_rng(13)
    # a different, deliberately non-top set per chunk (ascending, unique), different from chunk to chunk
    sets = np.stack([np.sort(rng.choice(M, size=k_eff, replace=False)) for _ in range(g.shape[0])]).astype(np.int32)
    out = orc.compress_chunks(g, m, s, rows, k, beta, forced_idx=sets, alpha=alpha)
    assert np.array_equal(out["idx"], sets)
    for c in range(g.shape[0]):
        B = (beta * m[c] + g[c]).reshape(rows, s)
        Q = scipy.fft.dctn(B, type=2, norm="ortho")
        assert np.max(np.abs(out["Q"][c].reshape(rows, s) - Q)) < 1e-12
        keep = np.zeros(M)
        keep[sets[c]] = Q.reshape(-1)[sets[c]]
        want = B - alpha * scipy.fft.idctn(keep.reshape(rows, s), type=2, norm="ortho")
        assert np.max(np.abs(out["m_new"][c].reshape(rows, s) - want)) < 1e-12
        assert np.max(np.abs(out["val"][c] - Q.reshape(-1)[sets[c]])) < 1e-12
    # and it is not what the free selection gives (the forced branch was really taken)
    free = orc.compress_chunks(g, m, s, rows, k, beta, alpha=alpha)
    assert not np.array_equal(free["idx"], sets)
    assert np.max(np.abs(free["m_new"] - out["m_new"])) > 1e-3


def test_forced_index_tensor_driver_walks_the_sets_chunk_by_chunk():
    # 2 x 3 chunk grid: a stride or ordering mistake in the per-chunk forced sets would pair a chunk with
    # its neighbour's set
    s, k, beta = 8, 4, 0.5
    rng = np.random.default_rng(14)
    g = rng.standard_normal((16, 24))
    m = rng.standard_normal((16, 24))
    M = s * s
    sets = np.stack([np.sort(rng.choice(M, size=k, replace=False)) for _ in range(6)]).astype(np.int32)
    out = orc.compress_tensor(g, m, s, k, beta, forced_idx=sets)
    assert np.array_equal(out["records"]["idx"], sets)
    for c in range(6):
        k0, k1 = divmod(c, 3)  # chunks row-major over the chunk grid
        B = beta * m[8 * k0:8 * k0 + 8, 8 * k1:8 * k1 + 8] + g[8 * k0:8 * k0 + 8, 8 * k1:8 * k1 + 8]
        Q = scipy.fft.dctn(B, type=2, norm="ortho")
        keep = np.zeros(M)
        keep[sets[c]] = Q.reshape(-1)[sets[c]]
        want = B - scipy.fft.idctn(keep.reshape(8, 8), type=2, norm="ortho")
        assert np.max(np.abs(out["m_new"][8 * k0:8 * k0 + 8, 8 * k1:8 * k1 + 8] - want)) < 1e-12
        assert np.max(np.abs(out["val64"][c] - Q.reshape(-1)[sets[c]])) < 1e-12
        assert np.array_equal(out["records"]["val"][c], Q.reshape(-1)[sets[c]].astype(np.float32))
    # 1-D tensor, three segments
    g1 = rng.standard_normal(24)
    m1 = rng.standard_normal(24)
    sets1 = np.stack([np.sort(rng.choice(8, size=3, replace=False)) for _ in range(3)]).astype(np.int32)
    out1 = orc.compress_tensor(g1, m1, 8, 3, beta, forced_idx=sets1)
    for c in range(3):
        b = beta * m1[8 * c:8 * c + 8] + g1[8 * c:8 * c + 8]
        q = scipy.fft.dct(b, type=2, norm="ortho")
        keep = np.zeros(8)
        keep[sets1[c]] = q[sets1[c]]
        assert np.max(np.abs(out1["m_new"][8 * c:8 * c + 8] - (b - scipy.fft.idct(keep, type=2, norm="ortho")))) < 1e-12
