"""numpy front-end of the fp64 CPU oracle (test infrastructure, not product code).

Compiles ``demo_oracle.c`` with gcc (``-O2 -fopenmp``, no fast-math) into
``liboracle_demo.so`` next to this file and exposes its entry points on numpy arrays.
Only ``tests/``, the smoke check and the benchmark's cpu-baseline leg may import this
module; the CUDA library never does.  Every function mirrors one routine of the C file,
which cites the passages of the paper it follows.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "demo_oracle.c")
_LIB = os.path.join(_HERE, "liboracle_demo.so")
_lock = threading.Lock()
_lib = None

RECORD_DTYPE = np.dtype([("idx", "<i4"), ("val", "<f4")])  # 8-byte payload record


def build(force: bool = False) -> str:
    """Compile the C oracle if the shared object is missing or older than the source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        cmd = ["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    with _lock:
        if _lib is None:
            build()
            lib = ctypes.CDLL(_LIB)
            c_dp = ctypes.POINTER(ctypes.c_double)
            c_ip = ctypes.POINTER(ctypes.c_int32)
            vp = ctypes.c_void_p
            i32, i64, f64 = ctypes.c_int, ctypes.c_int64, ctypes.c_double
            lib.oracle_dct_matrix.argtypes = [i32, c_dp]
            lib.oracle_dct_matrix.restype = None
            lib.oracle_block_extract.argtypes = [c_dp, i64, i32, i32, i64, i64, c_dp]
            lib.oracle_block_extract.restype = None
            lib.oracle_forward.argtypes = [i32, i32, c_dp, c_dp, c_dp]
            lib.oracle_forward.restype = None
            lib.oracle_inverse.argtypes = [i32, i32, c_dp, c_dp, c_dp]
            lib.oracle_inverse.restype = None
            lib.oracle_topk.argtypes = [i32, i32, c_dp, c_ip, c_dp, c_dp]
            lib.oracle_topk.restype = None
            lib.oracle_compress_chunks.argtypes = [i64, i32, i32, i32, f64, f64, c_dp, c_dp, c_ip, c_dp, c_ip,
                                                   c_dp, c_dp, c_dp, i32, c_dp]
            lib.oracle_compress_chunks.restype = None
            lib.oracle_compress_tensor.argtypes = [i32, i64, i64, i32, i32, f64, f64, c_dp, c_dp, c_ip, vp, c_dp,
                                                   c_dp, i32, c_dp]
            lib.oracle_compress_tensor.restype = i32
            lib.oracle_decode_chunks.argtypes = [i64, i32, i32, i32, i32, i32, i32, vp, c_dp, f64, f64, c_dp, c_dp, i32, c_dp]
            lib.oracle_decode_chunks.restype = None
            lib.oracle_decode_tensor.argtypes = [i32, i64, i64, i32, i32, i32, i32, i32, ctypes.POINTER(vp), c_dp, f64,
                                                 f64, c_dp, i32, c_dp]
            lib.oracle_decode_tensor.restype = i32
            lib.oracle_gram_schmidt.argtypes = [i32, c_dp, c_dp]
            lib.oracle_gram_schmidt.restype = i32
            lib.oracle_max_threads.argtypes = []
            lib.oracle_max_threads.restype = i32
            _lib = lib
    return _lib


def _dp(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def _ip(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_int32))


def _f64(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def _basis(basis, s):
    """(keep-alive array, pointer) of an optional s x s basis (rows = basis vectors); None = DCT."""
    if basis is None:
        return None, None
    b = _f64(basis)
    if b.shape != (s, s):
        raise ValueError("basis must be s x s")
    return b, _dp(b)


def gram_schmidt(G: np.ndarray) -> np.ndarray:
    """Rows of the square matrix G orthonormalised in order (Gram-Schmidt process)."""
    G = _f64(G)
    s = G.shape[0]
    if G.shape != (s, s):
        raise ValueError("G must be square")
    P = np.empty_like(G)
    if _load().oracle_gram_schmidt(s, _dp(G), _dp(P)) != 0:
        raise ValueError("G is singular to rounding")
    return P


def max_threads() -> int:
    return int(_load().oracle_max_threads())


def dct_matrix(s: int) -> np.ndarray:
    """Orthonormal DCT-II matrix C (s x s), C[u][n]."""
    C = np.empty((s, s), dtype=np.float64)
    _load().oracle_dct_matrix(s, _dp(C))
    return C


def block_extract(X: np.ndarray, s0: int, s1: int, k0: int, k1: int) -> np.ndarray:
    """Blocking operator: chunk (k0, k1) of shape s0 x s1 of the 2-D array X."""
    X = _f64(X)
    B = np.empty((s0, s1), dtype=np.float64)
    _load().oracle_block_extract(_dp(X), X.shape[1], s0, s1, k0, k1, _dp(B))
    return B


def forward(B: np.ndarray) -> np.ndarray:
    """Chunk DCT of one tile: (s, s) -> C B C^T, (s,) -> C b."""
    B = _f64(B)
    s = B.shape[-1]
    rows = 1 if B.ndim == 1 else B.shape[0]
    C = dct_matrix(s)
    Q = np.empty_like(B)
    _load().oracle_forward(s, rows, _dp(C), _dp(B), _dp(Q))
    return Q


def inverse(Q: np.ndarray) -> np.ndarray:
    """Inverse chunk DCT of one tile: (s, s) -> C^T Q C, (s,) -> C^T q."""
    Q = _f64(Q)
    s = Q.shape[-1]
    rows = 1 if Q.ndim == 1 else Q.shape[0]
    C = dct_matrix(s)
    R = np.empty_like(Q)
    _load().oracle_inverse(s, rows, _dp(C), _dp(Q), _dp(R))
    return R


def topk(Q: np.ndarray, k: int):
    """(ascending indices of the k_eff largest |Q|, ties to the lowest index; a_k; a_{k+1})."""
    Qf = _f64(Q).reshape(-1)
    M = Qf.size
    k_eff = min(k, M)
    idx = np.empty(k_eff, dtype=np.int32)
    a = ctypes.c_double()
    b = ctypes.c_double()
    _load().oracle_topk(M, k, _dp(Qf), _ip(idx), ctypes.byref(a), ctypes.byref(b))
    return idx, a.value, b.value


def compress_chunks(g, m, s: int, rows: int, k: int, beta: float, forced_idx=None, n_threads: int = 0,
                    alpha: float = 1.0, basis=None):
    """Independent chunks given as tiles [n, rows*s].

    Returns dict(Q [n,M], idx [n,k_eff] int32, val [n,k_eff] fp64, m_new [n,M], gap [n,2])."""
    g = _f64(g)
    m = _f64(m)
    M = rows * s
    n = g.size // M
    g = g.reshape(n, M)
    m = m.reshape(n, M)
    k_eff = min(k, M)
    Q = np.empty((n, M), dtype=np.float64)
    idx = np.empty((n, k_eff), dtype=np.int32)
    val = np.empty((n, k_eff), dtype=np.float64)
    m_new = np.empty((n, M), dtype=np.float64)
    gap = np.empty((n, 2), dtype=np.float64)
    fi = None
    if forced_idx is not None:
        fi = np.ascontiguousarray(forced_idx, dtype=np.int32).reshape(n, k_eff)
    _load().oracle_compress_chunks(n, s, rows, k, float(beta), float(alpha), _dp(g), _dp(m), _ip(fi) if fi is not None else None,
                                   _dp(Q), _ip(idx), _dp(val), _dp(m_new), _dp(gap), n_threads, _basis(basis, s)[1])
    return dict(Q=Q, idx=idx, val=val, m_new=m_new, gap=gap)


def compress_tensor(g, m, s: int, k: int, beta: float, forced_idx=None, n_threads: int = 0, alpha: float = 1.0,
                    basis=None):
    """One tensor (1-D or 2-D), one worker.  Returns dict(m_new, records [n_chunks,k_eff], val64, gap)."""
    g = _f64(g)
    m_new = _f64(m).copy()
    ndim = g.ndim
    n0, n1 = (1, g.shape[0]) if ndim == 1 else g.shape
    rows = s if ndim == 2 else 1
    M = rows * s
    k_eff = min(k, M)
    if n1 % s or (ndim == 2 and n0 % s):
        raise ValueError("tensor dims must be multiples of the chunk size")
    n_chunks = (n0 // rows) * (n1 // s)
    rec = np.zeros((n_chunks, k_eff), dtype=RECORD_DTYPE)
    val64 = np.empty((n_chunks, k_eff), dtype=np.float64)
    gap = np.empty((n_chunks, 2), dtype=np.float64)
    fi = None
    if forced_idx is not None:
        fi = np.ascontiguousarray(forced_idx, dtype=np.int32).reshape(n_chunks, k_eff)
    rc = _load().oracle_compress_tensor(ndim, n0, n1, s, k, float(beta), float(alpha), _dp(g), _dp(m_new),
                                        _ip(fi) if fi is not None else None, rec.ctypes.data_as(ctypes.c_void_p),
                                        _dp(val64), _dp(gap), n_threads, _basis(basis, s)[1])
    if rc != 0:
        raise ValueError("oracle_compress_tensor rejected the shape")
    return dict(m_new=m_new, records=rec, val64=val64, gap=gap)


AGG_SUM, AGG_MEAN, AGG_COUNT_MEAN = 0, 1, 2
PHI_SIGN, PHI_IDENTITY = 0, 1


def decode_chunks(records, x, s: int, rows: int, lr: float, wd: float, n_threads: int = 0, agg: int = 0, phi: int = 0,
                  basis=None):
    """records [W, n, k_eff] (RECORD_DTYPE), x [n, rows*s] -> dict(x_new [n,M], R [n,M])."""
    records = np.ascontiguousarray(records, dtype=RECORD_DTYPE)
    W, n, k_eff = records.shape
    M = rows * s
    x = _f64(x).reshape(n, M)
    x_new = np.empty_like(x)
    R = np.empty_like(x)
    _load().oracle_decode_chunks(n, s, rows, k_eff, W, agg, phi, records.ctypes.data_as(ctypes.c_void_p), _dp(x), float(lr),
                                 float(wd), _dp(x_new), _dp(R), n_threads, _basis(basis, s)[1])
    return dict(x_new=x_new, R=R)


def decode_tensor(payloads, x, s: int, k: int, lr: float, wd: float, n_threads: int = 0, agg: int = 0, phi: int = 0,
                  basis=None):
    """payloads: list over workers of [n_chunks, k_eff] record arrays for this tensor.

    Returns dict(x_new, R) with R the reconstructed global momentum of the tensor."""
    x_new = _f64(x).copy()
    ndim = x_new.ndim
    n0, n1 = (1, x_new.shape[0]) if ndim == 1 else x_new.shape
    W = len(payloads)
    keep = [np.ascontiguousarray(p, dtype=RECORD_DTYPE) for p in payloads]
    arr = (ctypes.c_void_p * W)(*[p.ctypes.data for p in keep])
    R = np.empty_like(x_new)
    rc = _load().oracle_decode_tensor(ndim, n0, n1, s, k, W, agg, phi, arr, _dp(x_new), float(lr), float(wd), _dp(R),
                                      n_threads, _basis(basis, s)[1])
    if rc != 0:
        raise ValueError("oracle_decode_tensor rejected the shape")
    return dict(x_new=x_new, R=R)
