"""Seeded synthetic workloads: shapes, hyper-parameters and value generators of the five benchmark
configurations.  This module serves both the CUDA path's tests/benchmark and the CPU oracle's
tests; it holds none of the method's arithmetic (no momentum update, DCT, top-k or update).

The paper trains OLMo-300M / OLMo-1B on a public corpus (Section 4); neither the models nor the
data are available here, so gradients are drawn from the distributions below with the same tensor
shapes, chunk size s, k and momentum decay as the paper's experiments.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Tuple

import torch

Shape = Tuple[int, ...]


@dataclass
class Workload:
    name: str
    shapes: List[Shape]
    chunk: int
    topk: int
    num_workers: int
    beta: float = 0.999
    lr: float = 1e-3
    weight_decay: float = 0.1
    grad_dtype: torch.dtype = torch.bfloat16
    grad_kind: str = "normal"  # normal | row_lognormal | tensor_scaled | student_t_ties
    grad_std: float = 1e-3
    steps: int = 1
    notes: str = ""
    tensor_names: List[str] = field(default_factory=list)

    @property
    def n_params(self) -> int:
        return sum(math.prod(s) for s in self.shapes)

    def n_chunks(self) -> int:
        s = self.chunk
        return sum(math.prod(d // s for d in shp) for shp in self.shapes)

    def records_per_worker(self) -> int:
        s = self.chunk
        tot = 0
        for shp in self.shapes:
            M = s * s if len(shp) == 2 else s
            tot += math.prod(d // s for d in shp) * min(self.topk, M)
        return tot


def _decoder_shapes(d_model: int, n_layers: int, d_ff: int, vocab: int, untied_head: bool):
    shapes, names = [], []
    for layer in range(n_layers):
        for nm in ("wq", "wk", "wv", "wo"):
            shapes.append((d_model, d_model))
            names.append("l%d.%s" % (layer, nm))
        shapes += [(d_ff, d_model), (d_ff, d_model), (d_model, d_ff)]
        names += ["l%d.gate" % layer, "l%d.up" % layer, "l%d.down" % layer]
        shapes += [(d_model,), (d_model,)]
        names += ["l%d.norm1" % layer, "l%d.norm2" % layer]
    shapes.append((vocab, d_model))
    names.append("embedding")
    if untied_head:
        shapes.append((d_model, vocab))
        names.append("head")
    return shapes, names


def tiny() -> Workload:
    return Workload("tiny", [(256, 512), (512,)], chunk=8, topk=4, num_workers=2, grad_dtype=torch.float32,
                    grad_kind="normal", grad_std=0.01, steps=3, tensor_names=["weight", "bias"],
                    notes="one fp32 weight 256x512 + bias 512, fp32 grads N(0, 0.01^2)")


def single_matrix() -> Workload:
    return Workload("single_8192", [(8192, 8192)], chunk=64, topk=32, num_workers=1, grad_kind="row_lognormal",
                    grad_std=1.0, steps=10, tensor_names=["matrix"],
                    notes="one 8192x8192 matrix, bf16 grads N(0,1) scaled per row by exp(N(0,1))")


def decoder_300m() -> Workload:
    shapes, names = _decoder_shapes(1024, 24, 4096, 50304, untied_head=False)
    return Workload("decoder_300m", shapes, chunk=64, topk=32, num_workers=8, grad_kind="tensor_scaled",
                    tensor_names=names, notes="300M-class decoder set, tied embedding, W=8")


def decoder_1b() -> Workload:
    shapes, names = _decoder_shapes(2048, 16, 8192, 50304, untied_head=True)
    return Workload("decoder_1b", shapes, chunk=64, topk=32, num_workers=16, grad_kind="tensor_scaled",
                    tensor_names=names, notes="1B-class decoder set, untied head, W=16")


def stress(chunk: int = 64, topk: int = 32, num_workers: int = 8, full_set: bool = True) -> Workload:
    if full_set:
        shapes, names = _decoder_shapes(2048, 16, 8192, 50304, untied_head=True)
    else:
        shapes, names = [], []
    shapes = shapes + [(4096, 4096)]
    names = names + ["stress_4096"]
    return Workload("stress_s%d_k%d_w%d%s" % (chunk, topk, num_workers, "" if full_set else "_matrix"), shapes,
                    chunk=chunk, topk=topk, num_workers=num_workers, grad_kind="student_t_ties",
                    tensor_names=names, notes="Student-t(3) * 1e-3 grads, 5% tie-maker chunks")


def by_name(name: str) -> Workload:
    table = {"tiny": tiny, "single_8192": single_matrix, "decoder_300m": decoder_300m, "decoder_1b": decoder_1b}
    if name in table:
        return table[name]()
    raise KeyError(name)


def small_decoder(d_model: int = 256, n_layers: int = 2, vocab: int = 1024, **kw) -> Workload:
    """A scaled-down decoder set (same tensor mix) for quick parity runs."""
    shapes, names = _decoder_shapes(d_model, n_layers, 4 * d_model, vocab, untied_head=True)
    args = dict(chunk=64, topk=32, num_workers=4, grad_kind="tensor_scaled")
    args.update(kw)
    return Workload("small_decoder", shapes, tensor_names=names, **args)


PARAM_SEED = 10_000
TENSOR_SCALE_SEED = 20_000
TIE_MASK_SEED = 30_000
ROW_FACTOR_SEED = 1
ROW_MASK_SEED = 40_000


def _gen(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def make_params(wl: Workload, device) -> List[torch.Tensor]:
    """Parameters ~ N(0, 0.02^2), fp32, seed PARAM_SEED, drawn in tensor order."""
    gen = _gen(device, PARAM_SEED)
    return [torch.randn(shp, generator=gen, device=device, dtype=torch.float32) * 0.02 for shp in wl.shapes]


def make_momentum(wl: Workload, device) -> List[torch.Tensor]:
    """Momentum starts at zero."""
    return [torch.zeros(shp, device=device, dtype=torch.float32) for shp in wl.shapes]


def tensor_scales(wl: Workload) -> List[float]:
    """Per-tensor gradient scale, log-uniform over [0.1, 10], shared by all workers."""
    gen = _gen("cpu", TENSOR_SCALE_SEED)
    u = torch.rand(len(wl.shapes), generator=gen, dtype=torch.float64)
    return [float(10.0 ** (2.0 * v - 1.0)) for v in u]


class GradStream:
    """Gradients of one worker: seed = worker index, drawn step-major then in tensor order."""

    def __init__(self, wl: Workload, worker: int, device):
        self.wl = wl
        self.worker = worker
        self.device = device
        self.gen = _gen(device, worker)
        self.scales = tensor_scales(wl) if wl.grad_kind == "tensor_scaled" else None
        self.row_factors = None
        if wl.grad_kind == "row_lognormal":
            rg = _gen(device, ROW_FACTOR_SEED)
            # one factor per row of a matrix, per element of a vector (its "rows" have one element)
            self.row_factors = [torch.exp(torch.randn((shp[0], 1) if len(shp) == 2 else (shp[0],), generator=rg, device=device))
                                for shp in wl.shapes]
        self.tie_gen = _gen(device, TIE_MASK_SEED + worker) if wl.grad_kind == "student_t_ties" else None
        self.tie_fraction = 0.05  # share of chunks replaced by tie-makers (student_t_ties)
        # Ablation: rows of the tensor named "embedding" that receive a gradient, per block of `chunk` rows
        # (only the tokens of a batch have a row); None = every row, the default of all configurations.
        self.embedding_active_rows = None
        self.row_gen = _gen(device, ROW_MASK_SEED + worker)

    def _draw(self, t: int, shp: Shape) -> torch.Tensor:
        wl = self.wl
        z = torch.randn(shp, generator=self.gen, device=self.device, dtype=torch.float32)
        if wl.grad_kind == "normal":
            return z * wl.grad_std
        if wl.grad_kind == "row_lognormal":
            return z * wl.grad_std * self.row_factors[t]
        if wl.grad_kind == "tensor_scaled":
            return z * (wl.grad_std * self.scales[t])
        if wl.grad_kind == "student_t_ties":
            chi = torch.zeros(shp, device=self.device, dtype=torch.float32)
            for _ in range(3):
                chi += torch.randn(shp, generator=self.gen, device=self.device, dtype=torch.float32) ** 2
            g = z / torch.sqrt(chi / 3.0) * wl.grad_std
            return self._tie_chunks(g, shp)
        raise ValueError(wl.grad_kind)

    def _tie_chunks(self, g: torch.Tensor, shp: Shape) -> torch.Tensor:
        """Replace a seeded 5% of the chunks by tiles that force ties in the top-k."""
        s = self.wl.chunk
        if len(shp) == 2:
            c0, c1 = shp[0] // s, shp[1] // s
            tiles = g.view(c0, s, c1, s).permute(0, 2, 1, 3)  # [c0, c1, s, s] view
        else:
            c0, c1 = 1, shp[0] // s
            tiles = g.view(1, c1, 1, s)
        pick = torch.rand((c0, c1), generator=self.tie_gen, device=self.device) < self.tie_fraction
        kind = torch.randint(0, 4, (c0, c1), generator=self.tie_gen, device=self.device)
        a = 1e-3
        sign = torch.where(torch.rand(tiles.shape, generator=self.tie_gen, device=self.device) < 0.5, -a, a)
        sym = 0.5 * (tiles + tiles.transpose(2, 3)) if len(shp) == 2 else tiles
        const = torch.where(torch.rand((c0, c1, 1, 1), generator=self.tie_gen, device=self.device) < 0.5, -a, a)
        out = tiles.clone()
        for kk, repl in enumerate((torch.zeros_like(tiles), const.expand_as(tiles), sym, sign)):
            sel = (pick & (kind == kk))[:, :, None, None]
            out = torch.where(sel, repl, out)
        if len(shp) == 2:
            return out.permute(0, 2, 1, 3).reshape(shp)
        return out.reshape(shp)

    def _mask_rows(self, g: torch.Tensor) -> torch.Tensor:
        """Keep `embedding_active_rows` seeded random rows in every block of `chunk` rows, zero the others."""
        s, r = self.wl.chunk, int(self.embedding_active_rows)
        blocks = g.shape[0] // s
        order = torch.rand((blocks, s), generator=self.row_gen, device=self.device).argsort(dim=1)
        keep = (order < r).reshape(-1, 1)
        return torch.where(keep, g, torch.zeros_like(g))

    def next(self) -> List[torch.Tensor]:
        out = []
        for t, shp in enumerate(self.wl.shapes):
            g = self._draw(t, shp)
            if self.embedding_active_rows is not None and t < len(self.wl.tensor_names) and \
                    self.wl.tensor_names[t] == "embedding":
                g = self._mask_rows(g)
            out.append(g.to(self.wl.grad_dtype))
        return out


def random_tensor(shape: Shape, seed: int, std: float, dtype: torch.dtype, device) -> torch.Tensor:
    """N(0, std^2) tensor of any shape from its own seed (tensors of order > 2, rectangular chunks)."""
    return (torch.randn(tuple(shape), generator=_gen(device, seed), device=device, dtype=torch.float32) * std).to(dtype)


def basis_gaussian(step: int, s: int) -> torch.Tensor:
    """s x s matrix of N(0,1) draws for the random orthonormal basis of one step; the seed is the step
    number, so every worker draws the same matrix (Section 4.2)."""
    gen = torch.Generator(device="cpu")
    gen.manual_seed(int(step))
    return torch.randn((s, s), generator=gen, dtype=torch.float32)
