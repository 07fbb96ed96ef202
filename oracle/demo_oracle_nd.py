"""fp64 CPU oracle for tensors of any order d with rectangular chunks (test infrastructure, not
product code; only ``tests/`` may import it, the CUDA library never does).

The appendix of the paper ("Multilinear Transforms and Chunk-wise Tensor Blocking") states the
method for a tensor of shape n_0 x ... x n_{d-1} cut into chunks of shape s_0 x ... x s_{d-1}
(n_i = c_i s_i): the blocking operator B, the multilinear product T(X; P_0, ..., P_{d-1}) with one
orthonormal matrix per axis (the DCT of dimension s_i), top-k per chunk, the residual and the
decode.  This module writes those definitions out with plain numpy in fp64, one chunk at a time, in
the paper's order; numpy's tensordot and sort serve as steps.  The square 2-D and the 1-D cases are
also covered by the C oracle (demo_oracle.c), which was written separately: the tests use the one to
check the other.

Conventions that the paper leaves open are those of the C oracle: records (int32 idx, fp32 val) with
idx the row-major position inside the chunk, ascending; exactly k_eff = min(k, M) records, ties at
the k-th magnitude to the lowest idx; chunks in row-major order over the chunk grid; sign(0) = 0.
"""
from __future__ import annotations

import numpy as np

RECORD_DTYPE = np.dtype([("idx", "<i4"), ("val", "<f4")])

AGG_SUM, AGG_MEAN, AGG_COUNT_MEAN = 0, 1, 2
PHI_SIGN, PHI_IDENTITY = 0, 1


def dct_matrix(s: int) -> np.ndarray:
    """Orthonormal DCT-II of dimension s: C[u][n] = a_u cos(pi (2n+1) u / (2s)), a_0 = sqrt(1/s),
    a_u = sqrt(2/s) otherwise (the unitary matrix of the appendix, P^T = P^-1)."""
    u = np.arange(s, dtype=np.float64)[:, None]
    n = np.arange(s, dtype=np.float64)[None, :]
    C = np.sqrt(2.0 / s) * np.cos(np.pi * (2.0 * n + 1.0) * u / (2.0 * s))
    C[0, :] = np.sqrt(1.0 / s)
    return C


def multilinear(X: np.ndarray, Ps) -> np.ndarray:
    """T(X; P_0, ..., P_{d-1}): out[i_0..i_{d-1}] = sum_j prod_k P_k[i_k][j_k] X[j_0..j_{d-1}]
    (appendix, definition of the multilinear product), one axis after the other."""
    Y = np.asarray(X, dtype=np.float64)
    if len(Ps) != Y.ndim:
        raise ValueError("one matrix per axis")
    for axis, P in enumerate(Ps):
        Y = np.moveaxis(np.tensordot(np.asarray(P, dtype=np.float64), Y, axes=([1], [axis])), 0, axis)
    return Y


def blocks(X: np.ndarray, chunk) -> np.ndarray:
    """Blocking operator: array [c_0, ..., c_{d-1}, s_0, ..., s_{d-1}] with
    out[k][j] = X[k_0 s_0 + j_0, ..., k_{d-1} s_{d-1} + j_{d-1}] (appendix, blocking operator)."""
    X = np.asarray(X)
    d = X.ndim
    if len(chunk) != d or any(n % s for n, s in zip(X.shape, chunk)):
        raise ValueError("every dimension must be a multiple of its chunk size")
    split = []
    for n, s in zip(X.shape, chunk):
        split += [n // s, s]
    return X.reshape(split).transpose(list(range(0, 2 * d, 2)) + list(range(1, 2 * d, 2)))


def unblocks(Bk: np.ndarray, shape) -> np.ndarray:
    """Inverse of `blocks`."""
    d = len(shape)
    order = []
    for i in range(d):
        order += [i, d + i]
    return np.ascontiguousarray(Bk.transpose(order)).reshape(shape)


def topk(q: np.ndarray, k: int):
    """(ascending indices of the k_eff largest |q|, ties to the lowest index; a_k; a_{k+1})."""
    q = np.asarray(q, dtype=np.float64).reshape(-1)
    M = q.size
    k_eff = min(k, M)
    mag = np.abs(q)
    order = np.lexsort((np.arange(M), -mag))  # by magnitude descending, then index ascending
    sel = np.sort(order[:k_eff]).astype(np.int32)
    a_k = mag[order[k_eff - 1]]
    a_k1 = mag[order[k_eff]] if k_eff < M else 0.0
    return sel, float(a_k), float(a_k1)


def compress_chunks(g, m, chunk, k: int, beta: float, forced_idx=None, alpha: float = 1.0):
    """Worker side of Algorithm 1 on n independent chunks given as rows [n, M] (M = prod(chunk),
    row-major inside the chunk): B = beta m + g; Q = T(B; C_0..C_{d-1}); keep the k_eff largest |Q|;
    m_new = B - alpha T(Q_kept; C_0^T..C_{d-1}^T).  `forced_idx` [n, k_eff] replaces the selection.

    Returns dict(Q [n,M], idx [n,k_eff] int32, val [n,k_eff] fp64, m_new [n,M], gap [n,2])."""
    chunk = tuple(int(s) for s in chunk)
    M = int(np.prod(chunk))
    g = np.asarray(g, dtype=np.float64).reshape(-1, M)
    m = np.asarray(m, dtype=np.float64).reshape(-1, M)
    n = g.shape[0]
    k_eff = min(k, M)
    Cs = [dct_matrix(s) for s in chunk]
    Cts = [C.T for C in Cs]
    Q = np.empty((n, M))
    idx = np.empty((n, k_eff), dtype=np.int32)
    val = np.empty((n, k_eff))
    m_new = np.empty((n, M))
    gap = np.empty((n, 2))
    for c in range(n):
        B = (beta * m[c] + g[c]).reshape(chunk)
        q = multilinear(B, Cs).reshape(-1)
        sel, a_k, a_k1 = topk(q, k)
        if forced_idx is not None:
            sel = np.asarray(forced_idx[c], dtype=np.int32)
        kept = np.zeros(M)
        kept[sel] = q[sel]
        Q[c], idx[c], val[c] = q, sel, q[sel]
        gap[c] = (a_k, a_k1)
        m_new[c] = (B - alpha * multilinear(kept.reshape(chunk), Cts)).reshape(-1)
    return dict(Q=Q, idx=idx, val=val, m_new=m_new, gap=gap)


def compress_tensor(g, m, chunk, k: int, beta: float, alpha: float = 1.0):
    """One tensor of any order, one worker.  Returns dict(m_new (tensor), records [n_chunks, k_eff],
    val64, gap); chunks in row-major order over the chunk grid."""
    g = np.asarray(g, dtype=np.float64)
    m = np.asarray(m, dtype=np.float64)
    chunk = tuple(int(s) for s in chunk)
    M = int(np.prod(chunk))
    gb = blocks(g, chunk)
    grid = gb.shape[: g.ndim]
    out = compress_chunks(gb.reshape(-1, M), blocks(m, chunk).reshape(-1, M), chunk, k, beta, alpha=alpha)
    rec = np.zeros(out["idx"].shape, dtype=RECORD_DTYPE)
    rec["idx"] = out["idx"]
    rec["val"] = out["val"].astype(np.float32)
    m_new = unblocks(out["m_new"].reshape(grid + chunk), g.shape)
    return dict(m_new=m_new, records=rec, val64=out["val"], gap=out["gap"])


def decode_chunks(records, x, chunk, lr: float, wd: float, agg: int = AGG_SUM, phi: int = PHI_SIGN):
    """Server side of Algorithm 1 on n chunks: records [W, n, k_eff], x [n, M].  S = sum over the
    workers in order of their records (mean: / W; count-normalised: / number of senders per
    coordinate, 0/0 = 0); R = T(S; C_0^T..C_{d-1}^T); x_new = x - lr (phi(R) + wd x)."""
    chunk = tuple(int(s) for s in chunk)
    M = int(np.prod(chunk))
    records = np.asarray(records, dtype=RECORD_DTYPE)
    W, n, _ = records.shape
    x = np.asarray(x, dtype=np.float64).reshape(n, M)
    Cts = [dct_matrix(s).T for s in chunk]
    x_new = np.empty_like(x)
    R = np.empty_like(x)
    for c in range(n):
        S = np.zeros(M)
        cnt = np.zeros(M)
        for w in range(W):
            np.add.at(S, records[w, c]["idx"], records[w, c]["val"].astype(np.float64))
            np.add.at(cnt, records[w, c]["idx"], 1.0)
        if agg == AGG_MEAN:
            S = S / W
        elif agg == AGG_COUNT_MEAN:
            S = np.where(cnt > 0, S / np.maximum(cnt, 1.0), 0.0)
        r = multilinear(S.reshape(chunk), Cts).reshape(-1)
        sg = r if phi == PHI_IDENTITY else np.sign(r)
        R[c] = r
        x_new[c] = x[c] - lr * (sg + wd * x[c])
    return dict(x_new=x_new, R=R)


def decode_tensor(payloads, x, chunk, lr: float, wd: float, agg: int = AGG_SUM, phi: int = PHI_SIGN):
    """payloads: list over workers of [n_chunks, k_eff] record arrays of this tensor."""
    x = np.asarray(x, dtype=np.float64)
    chunk = tuple(int(s) for s in chunk)
    M = int(np.prod(chunk))
    xb = blocks(x, chunk)
    grid = xb.shape[: x.ndim]
    out = decode_chunks(np.stack([np.asarray(p, dtype=RECORD_DTYPE) for p in payloads]), xb.reshape(-1, M), chunk, lr,
                        wd, agg=agg, phi=phi)
    return dict(x_new=unblocks(out["x_new"].reshape(grid + chunk), x.shape),
                R=unblocks(out["R"].reshape(grid + chunk), x.shape))
