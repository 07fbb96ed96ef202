"""Comparison harness: CUDA path (through the C ABI) against the fp64 CPU oracle, chunk by chunk.

Rules (written here once, used by every GPU parity test):
  * values / residual momentum / parameters:  |gpu - ref| <= 1e-5*|ref| + 1e-7*max(1, ||ref_chunk||_inf)
  * top-k index sets are compared bit for bit wherever the oracle's k-th and (k+1)-th magnitudes
    differ by more than 1e-5 relative (and the k-th is above the noise floor 1e-6*||Q||_inf);
    elsewhere the GPU's set must be a VALID top-k (selected magnitudes >= a_k(1-1e-5) - floor,
    unselected <= a_k(1+1e-5) + floor, ascending, unique, in range) and the oracle continues from
    the GPU's index set ("forced-index" residual);
  * decode is checked by feeding the GPU-written payload bytes to the oracle decode; the sign may
    differ only where |R| < 1e-6*max(1, ||R_chunk||_inf).
"""
from __future__ import annotations

import numpy as np
import torch

from oracle import demo_oracle as orc
from oracle import demo_oracle_nd as ond

RTOL = 1e-5
ATOL = 1e-7
GAP_RTOL = 1e-5
FLOOR_REL = 1e-6
SIGN_EXEMPT = 1e-6
# Momentum kept in the transform domain: what is compared is the inverse transform of stored coefficients that went
# through the twelve butterfly / rotation stages of a 2-D forward transform in fp32, not through one FMA and a sparse
# reconstruction; independent roundings add up as the root of the stage count (sqrt(12) = 3.5).
ATOL_M_DCT = 4e-7


def sample_chunk_ids(n_chunks: int, max_n: int, seed: int) -> np.ndarray:
    if n_chunks <= max_n:
        return np.arange(n_chunks, dtype=np.int64)
    rng = np.random.default_rng(seed)
    mid = rng.choice(np.arange(1, n_chunks - 1), size=max_n - 2, replace=False)
    return np.sort(np.concatenate([[0, n_chunks - 1], mid])).astype(np.int64)


def sample_chunk_fraction(n_chunks: int, denom: int, seed: int, min_n: int = 8) -> np.ndarray:
    """First and last chunk plus a seeded uniform sample, at least n_chunks / denom chunks in all (every chunk
    when the tensor has no more than min_n)."""
    want = max(min_n, -(-n_chunks // denom))
    return sample_chunk_ids(n_chunks, want, seed)


def gather_tiles(t: torch.Tensor, s: int, chunk_ids: np.ndarray) -> np.ndarray:
    """Tiles of the listed chunks (row-major chunk ids) as float64 [n, M]."""
    ids = torch.as_tensor(chunk_ids, device=t.device)
    if t.dim() == 2:
        c0, c1 = t.shape[0] // s, t.shape[1] // s
        v = t.view(c0, s, c1, s)
        tiles = v[ids // c1, :, ids % c1, :]  # [n, s, s]
    else:
        tiles = t.view(-1, s)[ids]
    return tiles.reshape(len(chunk_ids), -1).to(torch.float64).cpu().numpy()


def momentum_from_dct_tiles(tiles: np.ndarray, s: int) -> np.ndarray:
    """The momentum chunks behind buffers kept in the transform domain (demo_set_momentum_domain): a stored tile is the
    transposed coefficient tile, Q[u][v] = tile[v][u], and m = C^T Q C per chunk (fp64)."""
    C = orc.dct_matrix(s)
    Q = tiles.reshape(-1, s, s).transpose(0, 2, 1)
    return np.matmul(np.matmul(C.T, Q), C).reshape(tiles.shape[0], -1)


def gather_records(payload: torch.Tensor, first_record: int, k_eff: int, chunk_ids: np.ndarray) -> np.ndarray:
    """Records of the listed chunks of one tensor from a uint8 payload buffer -> [n, k_eff] records."""
    rec = payload.view(torch.int32).view(-1, 2)
    ids = torch.as_tensor(chunk_ids, device=payload.device)
    rows = first_record + ids[:, None] * k_eff + torch.arange(k_eff, device=payload.device)[None, :]
    got = rec[rows.reshape(-1)].cpu().numpy().reshape(len(chunk_ids), k_eff, 2)
    out = np.zeros((len(chunk_ids), k_eff), dtype=orc.RECORD_DTYPE)
    out["idx"] = got[:, :, 0]
    out["val"] = got[:, :, 1].copy().view(np.float32)
    return out


def _tol(ref: np.ndarray) -> np.ndarray:
    scale = np.maximum(1.0, np.max(np.abs(ref), axis=-1, keepdims=True))
    return RTOL * np.abs(ref) + ATOL * scale


class Report(dict):
    def add(self, key, n=1):
        self[key] = self.get(key, 0) + int(n)


def check_compress_chunks(g, m_before, m_after, rec_gpu, s, rows, k, beta, report: Report, what="", alpha=1.0,
                          basis=None, chunk_shape=None, m_atol=ATOL):
    """All arguments are per-chunk arrays of the same n chunks (float64 / records).  With `chunk_shape`
    (rectangular chunks of any order; s and rows unused) the reference is the N-D oracle."""
    if chunk_shape is not None:
        M = int(np.prod(chunk_shape))

        def oracle(gg, mm, forced_idx=None):
            return ond.compress_chunks(gg, mm, chunk_shape, k, beta, forced_idx=forced_idx, alpha=alpha)
    else:
        M = rows * s

        def oracle(gg, mm, forced_idx=None):
            return orc.compress_chunks(gg, mm, s, rows, k, beta, forced_idx=forced_idx, alpha=alpha, basis=basis)
    k_eff = min(k, M)
    n = g.shape[0]
    ref = oracle(g, m_before)
    Q = ref["Q"]
    qinf = np.max(np.abs(Q), axis=1)
    floor = FLOOR_REL * qinf
    a_k, a_k1 = ref["gap"][:, 0], ref["gap"][:, 1]
    pinned = (k_eff == M) | (((a_k - a_k1) > GAP_RTOL * a_k) & (a_k > floor))
    idx_gpu = rec_gpu["idx"].astype(np.int64)
    val_gpu = rec_gpu["val"].astype(np.float64)

    # structural checks on every chunk: in range, strictly ascending (hence unique)
    assert idx_gpu.min() >= 0 and idx_gpu.max() < M, what + ": record index out of range"
    if k_eff > 1:
        assert np.all(np.diff(idx_gpu, axis=1) > 0), what + ": record indices not strictly ascending"

    # pinned chunks: bit-exact index sets
    same = np.all(idx_gpu == ref["idx"], axis=1)
    bad = pinned & ~same
    assert not bad.any(), "%s: top-k index set differs on %d pinned chunk(s), first %d" % (
        what, bad.sum(), int(np.argmax(bad)))
    report.add("chunks", n)
    report.add("pinned", pinned.sum())
    report.add("unpinned", (~pinned).sum())
    report.add("unpinned_same_set", (~pinned & same).sum())

    # unpinned chunks with a different set: the GPU's set must be a valid top-k of the oracle's Q
    diff = np.nonzero(~same)[0]
    for c in diff:
        mag = np.abs(Q[c])
        sel = np.zeros(M, bool)
        sel[idx_gpu[c]] = True
        lo = a_k[c] * (1 - GAP_RTOL) - floor[c]
        hi = a_k[c] * (1 + GAP_RTOL) + floor[c]
        assert mag[sel].min() >= lo, what + ": chunk %d selected a coefficient below the threshold band" % c
        if k_eff < M:
            assert mag[~sel].max() <= hi, what + ": chunk %d missed a coefficient above the threshold band" % c

    # values at the GPU's own indices
    qref = np.take_along_axis(Q, idx_gpu, axis=1)
    scale = np.maximum(1.0, qinf)[:, None]
    err = np.abs(val_gpu - qref)
    okv = err <= RTOL * np.abs(qref) + ATOL * scale
    assert okv.all(), "%s: %d coefficient value(s) outside tolerance, max err %.3e (chunk %d)" % (
        what, (~okv).sum(), err.max(), int(np.argmax(err.max(axis=1))))
    report["max_val_err"] = max(report.get("max_val_err", 0.0), float(err.max()))
    report["max_val_err_unscaled_atol_viol"] = report.get("max_val_err_unscaled_atol_viol", 0) + int(
        (err > RTOL * np.abs(qref) + ATOL).sum())

    # residual momentum: oracle continued from the GPU's index set where the sets differ
    m_ref = ref["m_new"]
    if len(diff):
        forced = oracle(g[diff], m_before[diff], forced_idx=idx_gpu[diff].astype(np.int32))
        m_ref = m_ref.copy()
        m_ref[diff] = forced["m_new"]
    # the abs tolerance is scaled by the chunk's pre-subtraction magnitude (the fp32 rounding of
    # beta*m+g and of the reconstruction both scale with it)
    binf = np.maximum(1.0, np.maximum(np.max(np.abs(beta * m_before + g), axis=1), np.max(np.abs(m_ref), axis=1)))[:, None]
    errm = np.abs(m_after - m_ref)
    okm = errm <= RTOL * np.abs(m_ref) + m_atol * binf
    assert okm.all(), "%s: %d residual-momentum value(s) outside tolerance, max err %.3e (chunk %d)" % (
        what, (~okm).sum(), errm.max(), int(np.argmax(errm.max(axis=1))))
    report["max_m_err"] = max(report.get("max_m_err", 0.0), float(errm.max()))
    return ref


def check_decode_chunks(recs_gpu, x_before, x_after, s, rows, lr, wd, report: Report, what="", agg=0, phi=0,
                         basis=None, chunk_shape=None):
    """recs_gpu [W, n, k_eff] GPU-written records; x_* float64 [n, M]."""
    if chunk_shape is not None:
        ref = ond.decode_chunks(recs_gpu, x_before, chunk_shape, lr, wd, agg=agg, phi=phi)
    else:
        ref = orc.decode_chunks(recs_gpu, x_before, s, rows, lr, wd, agg=agg, phi=phi, basis=basis)
    R = ref["R"]
    if phi == orc.PHI_IDENTITY:
        # no sign decision: the update is linear in R; the tolerance follows R's fp32 rounding
        x_ref = ref["x_new"]
        rinf = np.maximum(1.0, np.max(np.abs(R), axis=1, keepdims=True))
        tol = RTOL * np.abs(x_ref) + ATOL * np.maximum(1.0, np.max(np.abs(x_ref), axis=1, keepdims=True)) + lr * (
            RTOL * np.abs(R) + ATOL * rinf)
        ok = np.abs(x_after - x_ref) <= tol
        assert ok.all(), "%s: %d parameter(s) outside tolerance (identity update)" % (what, (~ok).sum())
        report.add("decode_chunks", x_before.shape[0])
        return ref
    rinf = np.maximum(1.0, np.max(np.abs(R), axis=1, keepdims=True))
    exempt = np.abs(R) < SIGN_EXEMPT * rinf
    x_ref = ref["x_new"]
    tol = RTOL * np.abs(x_ref) + ATOL * np.maximum(1.0, np.max(np.abs(x_ref), axis=1, keepdims=True))
    ok = np.abs(x_after - x_ref) <= tol
    # where the reconstructed momentum is within rounding of zero any of the three signs is legal
    if (~ok & exempt).any():
        alt = np.zeros_like(ok)
        for sg in (-1.0, 0.0, 1.0):
            alt |= np.abs(x_after - (x_before - lr * (sg + wd * x_before))) <= tol
        ok = ok | (exempt & alt)
    assert ok.all(), "%s: %d parameter(s) outside tolerance (sign or value), first chunk %d" % (
        what, (~ok).sum(), int(np.argmax((~ok).any(axis=1))))
    report.add("decode_chunks", x_before.shape[0])
    report.add("sign_exempt", exempt.sum())
    # sign bit-exactness outside the exemption, recovered from the update itself
    sg_gpu = np.rint((x_before * (1.0 - lr * wd) - x_after) / lr)
    mism = (sg_gpu != np.sign(R)) & ~exempt
    assert not mism.any(), what + ": sign mismatch outside the exemption band"
    return ref


class Runner:
    """Drives a workload through the C ABI and checks sampled (or all) chunks every step."""

    def __init__(self, wl, device="cuda", max_chunks=256, path=None, seed=0, alpha=None, agg=0, phi=0, basis=None,
                 gauss=None, momentum_domain=None):
        import paper_2411_19870_b200 as demo
        from paper_2411_19870_b200 import inputs

        self.wl, self.device = wl, torch.device(device)
        self.demo = demo
        gd = demo.DEMO_BF16 if wl.grad_dtype == torch.bfloat16 else demo.DEMO_F32
        self.tr = demo.DemoTransform(wl.shapes, chunk=wl.chunk, topk=wl.topk, beta=wl.beta, lr=wl.lr,
                                     weight_decay=wl.weight_decay, num_workers=wl.num_workers, grad_dtype=gd,
                                     device=self.device.index or 0)
        if path is not None:
            self.tr.set_path(path)
        # momentum buffers of 2-D tensors in the transform domain: the oracle sees the momentum they stand for
        self.mom_dct = bool(momentum_domain)
        if momentum_domain is not None:
            self.tr.set_momentum_domain(momentum_domain)
        self.agg, self.phi = agg, phi
        if agg or phi:
            self.tr.set_decode_mode(agg, phi)
        # other bases: `basis` (s x s, rows = vectors) is handed to both sides; `gauss` is orthonormalised
        # by each side with its own Gram-Schmidt
        self.basis = None
        self.set_basis(basis, gauss)
        self.alpha = 1.0
        if alpha is not None:
            self.tr.set_alpha(alpha)
            self.alpha = float(np.float32(alpha))
        self.params = inputs.make_params(wl, self.device)
        self.mom = [inputs.make_momentum(wl, self.device) for _ in range(wl.num_workers)]
        self.streams = [inputs.GradStream(wl, w, self.device) for w in range(wl.num_workers)]
        self.payloads = [torch.zeros(self.tr.payload_bytes, dtype=torch.uint8, device=self.device)
                         for _ in range(wl.num_workers)]
        self.layout = [self.tr.payload_layout(t) for t in range(len(wl.shapes))]
        self.ids = [sample_chunk_ids(self.layout[t][1], max_chunks, seed + t) for t in range(len(wl.shapes))]
        self.report = Report()
        # fp32 copies of the scalars, as the library sees them
        self.beta = float(np.float32(wl.beta))
        self.lr = float(np.float32(wl.lr))
        self.wd = float(np.float32(wl.weight_decay))

    def set_basis(self, basis=None, gauss=None):
        if gauss is not None:
            g32 = np.ascontiguousarray(gauss, dtype=np.float32)
            self.tr.set_basis_gaussian(torch.from_numpy(g32))
            self.basis = orc.gram_schmidt(g32.astype(np.float64))
        elif basis is not None:
            b32 = np.ascontiguousarray(basis, dtype=np.float32)
            self.tr.set_basis(torch.from_numpy(b32))
            self.basis = b32.astype(np.float64)
        else:
            self.tr.set_basis(None)
            self.basis = None

    def momentum_tiles(self, w, t):
        tiles = gather_tiles(self.mom[w][t], self.wl.chunk, self.ids[t])
        if self.mom_dct and len(self.wl.shapes[t]) == 2:
            tiles = momentum_from_dct_tiles(tiles, self.wl.chunk)
        return tiles

    def step(self, check=True, grads=None, workers=None, invariants=False):
        """One optimizer step.  `workers`: the workers whose compress call is compared with the oracle (default:
        all); the decode is compared on the payloads of every worker either way.  `invariants`: also check the
        whole-tensor properties (every chunk, no oracle) of every worker's compress call."""
        wl, s = self.wl, self.wl.chunk
        T = len(wl.shapes)
        for w in range(wl.num_workers):
            g = grads[w] if grads is not None else self.streams[w].next()
            check_w = check and (workers is None or w in workers)
            if invariants:
                energy = [tensor_energy(self.beta, self.mom[w][t], g[t]) for t in range(T)]
            if check_w:
                before = [self.momentum_tiles(w, t) for t in range(T)]
            self.tr.compress(w, g, self.mom[w], self.payloads[w])
            if invariants:
                self.report.add("invariant_records", check_whole_tensor_invariants(
                    self.payloads[w], self.layout, wl.shapes, s, energy, self.mom[w], what="worker %d" % w))
            if check_w:
                for t in range(T):
                    rows = s if len(wl.shapes[t]) == 2 else 1
                    first, _, k_eff = self.layout[t]
                    check_compress_chunks(
                        gather_tiles(g[t], s, self.ids[t]), before[t], self.momentum_tiles(w, t),
                        gather_records(self.payloads[w], first, k_eff, self.ids[t]), s, rows, wl.topk, self.beta,
                        self.report, what="compress w%d t%d" % (w, t), alpha=self.alpha, basis=self.basis,
                        m_atol=ATOL_M_DCT if (self.mom_dct and rows > 1) else ATOL)
        if check:
            xb = [gather_tiles(self.params[t], s, self.ids[t]) for t in range(T)]
        self.tr.decode_apply(self.payloads, self.params)
        if check:
            for t in range(T):
                rows = s if len(wl.shapes[t]) == 2 else 1
                first, _, k_eff = self.layout[t]
                recs = np.stack([gather_records(self.payloads[w], first, k_eff, self.ids[t])
                                 for w in range(wl.num_workers)])
                check_decode_chunks(recs, xb[t], gather_tiles(self.params[t], s, self.ids[t]), s, rows, self.lr,
                                    self.wd, self.report, what="decode t%d" % t, agg=self.agg, phi=self.phi, basis=self.basis)
        st = self.tr.device_status()
        assert st == 0, "device status %d (%s)" % (st, self.demo.demo_status_string(st))

    def close(self):
        self.tr.close()


class NdRunner:
    """Tensors of any order with rectangular chunks (demo_init_nd) against the N-D oracle, every chunk of
    every tensor, every step."""

    def __init__(self, shapes, chunk_shapes, topk, num_workers=2, grad_dtype=torch.bfloat16, beta=0.999, lr=1e-3,
                 weight_decay=0.1, grad_std=1e-3, seed=0, alpha=None, agg=0, phi=0, device="cuda"):
        import paper_2411_19870_b200 as demo
        from paper_2411_19870_b200 import inputs

        self.demo, self.inputs = demo, inputs
        self.shapes = [tuple(s) for s in shapes]
        self.chunks = [tuple(c) for c in chunk_shapes]
        self.k, self.W, self.gdtype, self.grad_std, self.seed = topk, num_workers, grad_dtype, grad_std, seed
        self.device = torch.device(device)
        gd = demo.DEMO_BF16 if grad_dtype == torch.bfloat16 else demo.DEMO_F32
        self.tr = demo.DemoTransform(self.shapes, topk=topk, beta=beta, lr=lr, weight_decay=weight_decay,
                                     num_workers=num_workers, grad_dtype=gd, device=self.device.index or 0,
                                     chunk_shapes=self.chunks)
        self.agg, self.phi = agg, phi
        if agg or phi:
            self.tr.set_decode_mode(agg, phi)
        self.alpha = 1.0
        if alpha is not None:
            self.tr.set_alpha(alpha)
            self.alpha = float(np.float32(alpha))
        self.params = [inputs.random_tensor(s, inputs.PARAM_SEED + t, 0.02, torch.float32, self.device)
                       for t, s in enumerate(self.shapes)]
        self.mom = [[torch.zeros(s, dtype=torch.float32, device=self.device) for s in self.shapes]
                    for _ in range(num_workers)]
        self.payloads = [torch.zeros(self.tr.payload_bytes, dtype=torch.uint8, device=self.device)
                         for _ in range(num_workers)]
        self.layout = [self.tr.payload_layout(t) for t in range(len(self.shapes))]
        self.report = Report()
        self.beta, self.lr, self.wd = float(np.float32(beta)), float(np.float32(lr)), float(np.float32(weight_decay))
        self.step_no = 0

    def _tiles(self, t, tensor):
        M = int(np.prod(self.chunks[t]))
        return ond.blocks(tensor.to(torch.float64).cpu().numpy(), self.chunks[t]).reshape(-1, M)

    def _records(self, w, t):
        first, n_chunks, k_eff = self.layout[t]
        return gather_records(self.payloads[w], first, k_eff, np.arange(n_chunks, dtype=np.int64))

    def step(self):
        T = len(self.shapes)
        for w in range(self.W):
            g = [self.inputs.random_tensor(s, self.seed + 1000 * self.step_no + 100 * w + t, self.grad_std, self.gdtype,
                                           self.device) for t, s in enumerate(self.shapes)]
            before = [self._tiles(t, self.mom[w][t]) for t in range(T)]
            self.tr.compress(w, g, self.mom[w], self.payloads[w])
            for t in range(T):
                M = int(np.prod(self.chunks[t]))
                assert self.layout[t][2] == min(self.k, M)
                check_compress_chunks(self._tiles(t, g[t]), before[t], self._tiles(t, self.mom[w][t]), self._records(w, t),
                                      0, 0, self.k, self.beta, self.report, what="nd compress w%d t%d" % (w, t),
                                      alpha=self.alpha, chunk_shape=self.chunks[t])
        xb = [self._tiles(t, self.params[t]) for t in range(T)]
        self.tr.decode_apply(self.payloads, self.params)
        for t in range(T):
            recs = np.stack([self._records(w, t) for w in range(self.W)])
            check_decode_chunks(recs, xb[t], self._tiles(t, self.params[t]), 0, 0, self.lr, self.wd, self.report,
                                what="nd decode t%d" % t, agg=self.agg, phi=self.phi, chunk_shape=self.chunks[t])
        st = self.tr.device_status()
        assert st == 0, "device status %d (%s)" % (st, self.demo.demo_status_string(st))
        self.step_no += 1

    def close(self):
        self.tr.close()


# ---------------------------------------------------------------------------------------------------------
# Whole-tensor properties that hold at any size, evaluated on the device over EVERY chunk (no oracle call):
#   * every record index lies in its chunk and the indices of a chunk are strictly ascending (exactly k_eff
#     distinct coefficients per chunk, Section 2.1 "Top-k Sparsification");
#   * energy split of an orthonormal transform: ||m_new||^2 = ||beta m + g||^2 - sum val^2 per tensor
#     (Parseval; the residual is B minus the kept coefficients' reconstruction).
# ---------------------------------------------------------------------------------------------------------
def tensor_energy(beta: float, m: torch.Tensor, g: torch.Tensor) -> float:
    """sum (beta m + g)^2 of one tensor, accumulated in fp64 slice by slice (bounded temporary memory)."""
    tot = 0.0
    mf, gf = m.reshape(-1), g.reshape(-1)
    step = 1 << 26
    for i in range(0, mf.numel(), step):
        b = torch.add(gf[i:i + step].double(), mf[i:i + step].double(), alpha=beta)
        tot += float(b.pow(2).sum().item())
    return tot


def sum_squares(t: torch.Tensor) -> float:
    tot = 0.0
    f = t.reshape(-1)
    step = 1 << 26
    for i in range(0, f.numel(), step):
        tot += float(f[i:i + step].double().pow(2).sum().item())
    return tot


def check_whole_tensor_invariants(payload: torch.Tensor, layout, shapes, chunk: int, energy_before, mom_after,
                                  what: str = "", rtol: float = 1e-5) -> int:
    """payload: one worker's uint8 buffer; layout[t] = (first_record, n_chunks, k_eff); energy_before[t] =
    tensor_energy(...) taken before the compress call; mom_after: that worker's momentum tensors after it.
    Returns the number of records seen."""
    rec = payload.view(torch.int32).view(-1, 2)
    seen = 0
    for t, shp in enumerate(shapes):
        first, n_chunks, k_eff = layout[t]
        M = chunk * chunk if len(shp) == 2 else chunk
        rr = rec[first:first + n_chunks * k_eff].view(n_chunks, k_eff, 2)
        idx = rr[:, :, 0]
        assert int(idx.min().item()) >= 0 and int(idx.max().item()) < M, "%s t%d: record index out of range" % (what, t)
        if k_eff > 1:
            assert bool(torch.all(idx[:, 1:] > idx[:, :-1]).item()), "%s t%d: indices not strictly ascending" % (what, t)
        val2 = float(rr[:, :, 1].contiguous().view(torch.float32).double().pow(2).sum().item())
        lhs = sum_squares(mom_after[t])
        rhs = energy_before[t] - val2
        assert abs(lhs - rhs) <= rtol * max(energy_before[t], 1e-300), "%s t%d: energy identity off by %.3e of %.3e" % (
            what, t, abs(lhs - rhs), energy_before[t])
        seen += n_chunks * k_eff
    assert seen == rec.shape[0], "%s: payload holds %d records, the layout accounts for %d" % (what, rec.shape[0], seen)
    return seen
