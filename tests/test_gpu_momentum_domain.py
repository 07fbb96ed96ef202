"""Momentum kept in the transform domain (demo_set_momentum_domain, an opt-in re-statement of Algorithm 1 that the
paper does not have): the buffers of 2-D tensors hold the transposed DCT tiles of the momentum.  The oracle knows
nothing of this; every step the test turns the stored tiles back into the momentum they stand for with an fp64
inverse transform and compares records and new momentum with the oracle's step from that momentum."""
import numpy as np
import pytest
import torch

import paper_2411_19870_b200 as demo
from paper_2411_19870_b200 import inputs
from tests import parity

pytestmark = pytest.mark.gpu

DCT = demo.DEMO_MOMENTUM_DCT


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_small_decoder_step_locked(dtype):
    """2-D and 1-D tensors, k = 32, W = 4, five steps, every chunk."""
    wl = inputs.small_decoder(grad_dtype=dtype)
    r = parity.Runner(wl, max_chunks=10**9, momentum_domain=DCT)
    for _ in range(5):
        r.step()
    assert r.report["pinned"] > 0.98 * r.report["chunks"]
    r.close()


@pytest.mark.parametrize("k,alpha", [(1, None), (8, 0.5), (64, None), (100, 0.25), (256, None), (700, None), (4096, None)])
def test_topk_range_and_partial_subtraction(k, alpha):
    """k from 1 to the whole chunk (the selection's ordinary path, its candidate path for k > 64, the radix path) and
    alpha < 1 (what stays of a transmitted coefficient is q - alpha q)."""
    wl = inputs.small_decoder(topk=k, num_workers=2)
    r = parity.Runner(wl, max_chunks=60, alpha=alpha, momentum_domain=DCT)
    for _ in range(3):
        r.step()
    r.close()


def test_ties_and_heavy_tails_take_the_out_of_line_selection():
    wl = inputs.stress(num_workers=2, full_set=False)
    r = parity.Runner(wl, max_chunks=200, momentum_domain=DCT)
    for _ in range(3):
        r.step()
    r.close()


def test_degenerate_chunks():
    """Zero gradient on zero momentum (records 0 .. k-1 with value 0), a constant tile (one coefficient), a tile of
    rank one."""
    s, k = 64, 32
    wl = inputs.Workload("degenerate", [(2 * s, 2 * s)], chunk=s, topk=k, num_workers=1, grad_dtype=torch.float32)
    r = parity.Runner(wl, max_chunks=10**9, momentum_domain=DCT)
    g = torch.zeros(2 * s, 2 * s, device="cuda")
    g[:s, s:] = 0.25
    u = torch.linspace(-1, 1, s, device="cuda")
    g[s:, :s] = u[:, None] * torch.cos(3 * u)[None, :]
    g[s:, s:] = torch.randn(s, s, device="cuda", generator=torch.Generator("cuda").manual_seed(5))
    for _ in range(2):
        r.step(grads=[[g]])
    rec = parity.gather_records(r.payloads[0], 0, k, np.arange(4))
    assert np.array_equal(rec["idx"][0], np.arange(k)) and not rec["val"][0].any()
    assert rec["idx"][1][0] == 0 and abs(rec["val"][1][0]) > 1.0
    r.close()


def test_same_records_as_the_spatial_momentum_over_steps():
    """Both representations run side by side on the same gradients: after five steps (no oracle in between) the
    index sets agree on all chunks but near-ties and the values to fp32 rounding."""
    wl = inputs.small_decoder(num_workers=1)
    a = parity.Runner(wl, max_chunks=10**9)
    b = parity.Runner(wl, max_chunks=10**9, momentum_domain=DCT)
    for _ in range(5):
        g = [a.streams[0].next()]
        a.step(check=False, grads=g)
        b.step(check=False, grads=g)
    pa = a.payloads[0].view(torch.int32).view(-1, 2)
    pb = b.payloads[0].view(torch.int32).view(-1, 2)
    same = (pa[:, 0] == pb[:, 0])
    assert same.float().mean().item() > 0.995
    va, vb = pa[:, 1].view(torch.float32)[same], pb[:, 1].view(torch.float32)[same]
    assert torch.allclose(va, vb, rtol=1e-4, atol=1e-6 * va.abs().max().item())
    a.close()
    b.close()


def test_refused_where_no_kernel_implements_it():
    wl = inputs.small_decoder(chunk=32)
    r = parity.Runner(wl, max_chunks=4)
    with pytest.raises(demo.DemoError):
        r.tr.set_momentum_domain(DCT)
    r.close()
    tr = demo.DemoTransform([(64, 128)], topk=8, beta=0.9, lr=1e-3, weight_decay=0.0, num_workers=1,
                            chunk_shapes=[(32, 64)])
    with pytest.raises(demo.DemoError):
        tr.set_momentum_domain(DCT)
    tr.close()
    # the generic kernels and a caller-supplied basis keep the momentum itself: compress refuses, nothing is written
    wl = inputs.small_decoder(num_workers=1)
    r = parity.Runner(wl, max_chunks=4, momentum_domain=DCT)
    g = [r.streams[0].next()]
    r.tr.set_path(demo.DEMO_PATH_GENERIC)
    before = [m.clone() for m in r.mom[0]]
    with pytest.raises(demo.DemoError):
        r.tr.compress(0, g[0], r.mom[0], r.payloads[0])
    r.tr.set_path(demo.DEMO_PATH_AUTO)
    r.set_basis(basis=np.eye(64, dtype=np.float32))
    with pytest.raises(demo.DemoError):
        r.tr.compress(0, g[0], r.mom[0], r.payloads[0])
    assert all(torch.equal(x, y) for x, y in zip(before, r.mom[0]))
    r.set_basis(None)
    r.tr.set_momentum_domain(demo.DEMO_MOMENTUM_SPATIAL)
    r.mom_dct = False  # (the buffers are still all zero: no conversion needed)
    r.step(grads=g)
    r.close()
