"""GPU parity of the kernels for tensors of any order with rectangular chunks (demo_init_nd) against the
N-D oracle, every chunk of every tensor (rules in tests/parity.py)."""
import numpy as np
import pytest
import torch

import paper_2411_19870_b200 as demo
from paper_2411_19870_b200 import inputs
from tests import parity

pytestmark = pytest.mark.gpu


def test_blocking_example_of_the_paper_128x512_in_16x32():
    """The appendix's worked example: a 128 x 512 matrix in 16 x 32 blocks (8 x 16 grid)."""
    r = parity.NdRunner([(128, 512)], [(16, 32)], topk=8, num_workers=2)
    assert r.layout[0] == (0, 8 * 16, 8)
    for _ in range(3):
        r.step()
    assert r.report["chunks"] == 3 * 2 * 128 and r.report["pinned"] > 0.95 * r.report["chunks"]
    r.close()


@pytest.mark.parametrize("shapes,chunks,k", [
    ([(8, 12, 20), (64,)], [(4, 3, 5), (16,)], 7),                 # order 3 with odd extents + a vector
    ([(4, 6, 8, 16)], [(2, 3, 4, 8)], 20),                         # order 4
    ([(96, 40), (6, 64, 64)], [(32, 8), (1, 64, 64)], 32),         # rectangular + a stack of 64 x 64 tiles
    ([(256, 128), (64, 48)], [(128, 128), (32, 16)], 64),              # the largest chunk (16384 elements); the small
                                                                   # rectangular tensor keeps the context on the N-D kernels
    ([(5, 7, 3)], [(1, 1, 1)], 1),                                 # every extent 1: the identity transform
    ([(128, 6)], [(128, 1)], 9),                                   # a column chunk
])
def test_shapes_and_chunks(shapes, chunks, k):
    r = parity.NdRunner(shapes, chunks, topk=k, num_workers=3, grad_std=1.0)
    for _ in range(2):
        r.step()
    assert r.report["chunks"] > 0
    r.close()


def test_lossless_when_k_exceeds_the_chunk():
    """k > M keeps every coefficient: the residual is fp32 rounding of a round trip, a few ulp of the
    chunk's magnitude (hence gradients of size 1e-3, where that sits below the absolute tolerance)."""
    r = parity.NdRunner([(30, 21)], [(3, 7)], topk=100, num_workers=3, grad_std=1e-3)
    assert r.layout[0] == (0, 30, 21)
    for _ in range(2):
        r.step()
    for w in range(3):
        assert float(r.mom[w][0].abs().max()) < 1e-8
    r.close()


@pytest.mark.parametrize("agg,phi", [(1, 0), (2, 0), (0, 1), (2, 1)])
def test_aggregation_phi_and_alpha(agg, phi):
    r = parity.NdRunner([(16, 12, 10)], [(8, 4, 5)], topk=12, num_workers=4, agg=agg, phi=phi, alpha=0.2,
                        grad_dtype=torch.float32)
    for _ in range(3):
        r.step()
    r.close()


def test_square_chunks_match_the_square_chunk_context():
    """Tensors with equal chunk extents inside an N-D context (a rectangular third tensor keeps it on the dense
    per-axis kernels): same records per tensor as demo_init through its dense kernels -- index sets bit for bit,
    values / momenta / parameters equal to fp32 rounding of a different summation order."""
    dev = torch.device("cuda")
    shapes, s, k, W = [(128, 192), (256,)], 32, 17, 2
    kw = dict(topk=k, beta=0.9, lr=1e-3, weight_decay=0.1, num_workers=W, grad_dtype=demo.DEMO_F32)
    a = demo.DemoTransform(shapes, chunk=s, **kw)
    a.set_path(demo.DEMO_PATH_GENERIC)
    shapes_b = shapes + [(64, 48)]
    b = demo.DemoTransform(shapes_b, chunk_shapes=[(s, s), (s,), (16, 8)], **kw)
    with pytest.raises(demo.DemoError):
        b.set_basis(torch.eye(s))              # an N-D context: one basis per chunk extent, only the DCT
    assert [a.payload_layout(t) for t in range(2)] == [b.payload_layout(t) for t in range(2)]
    n_rec = a.payload_bytes // 8
    state = []
    for tr, shp in ((a, shapes), (b, shapes_b)):
        x = [inputs.random_tensor(sh, 5 + t, 0.02, torch.float32, dev) for t, sh in enumerate(shp)]
        mom = [[torch.zeros(sh, device=dev) for sh in shp] for _ in range(W)]
        pay = [torch.zeros(tr.payload_bytes, dtype=torch.uint8, device=dev) for _ in range(W)]
        for step in range(3):
            for w in range(W):
                g = [inputs.random_tensor(sh, 100 * step + 10 * w + t, 1.0, torch.float32, dev) for t, sh in enumerate(shp)]
                tr.compress(w, g, mom[w], pay[w])
            tr.decode_apply(pay, x)
        assert tr.device_status() == 0
        state.append((pay, mom, x))
    for w in range(W):
        ia = state[0][0][w].view(torch.int32).view(-1, 2)[:n_rec]
        ib = state[1][0][w].view(torch.int32).view(-1, 2)[:n_rec]
        assert torch.equal(ia[:, 0], ib[:, 0])  # index sets bit for bit
        va = state[0][0][w].view(torch.float32).view(-1, 2)[:n_rec, 1]
        vb = state[1][0][w].view(torch.float32).view(-1, 2)[:n_rec, 1]
        assert torch.allclose(va, vb, rtol=1e-5, atol=1e-6)  # summation orders differ
        for t in range(len(shapes)):
            assert torch.allclose(state[0][1][w][t], state[1][1][w][t], rtol=1e-5, atol=1e-6)
    for t in range(len(shapes)):
        assert torch.allclose(state[0][2][t], state[1][2][t], rtol=1e-5, atol=1e-6)
    a.close()
    b.close()


@pytest.mark.parametrize("s,k", [(64, 32), (128, 40), (32, 2000)])
def test_square_chunk_descriptors_take_the_square_chunk_kernels(s, k):
    """demo_init_nd with s x s tiles of the last two axes / length-s segments of the last axis everywhere (leading
    chunk extents 1) is demo_init on the flattened tensors: same kernels, so every output is bit for bit the same,
    and what only that kind of context offers (a caller-supplied basis) is accepted."""
    dev = torch.device("cuda")
    nd_shapes = [(2 * s, 3 * s), (3, 2 * s, 2 * s), (4 * s,), (5, 2 * s)]
    nd_chunks = [(s, s), (1, s, s), (s,), (1, s)]
    flat_shapes = [(2 * s, 3 * s), (6 * s, 2 * s), (4 * s,), (10 * s,)]
    W = 2
    kw = dict(beta=0.999, lr=1e-3, weight_decay=0.1, num_workers=W)
    a = demo.DemoTransform(flat_shapes, chunk=s, topk=min(k, s * s), **kw)
    b = demo.DemoTransform(nd_shapes, chunk_shapes=nd_chunks, topk=k, **kw)
    assert a.payload_bytes == b.payload_bytes
    assert [a.payload_layout(t) for t in range(4)] == [b.payload_layout(t) for t in range(4)]
    out = []
    for tr, shp in ((a, flat_shapes), (b, nd_shapes)):
        x = [inputs.random_tensor(sh, 5 + t, 0.02, torch.float32, dev) for t, sh in enumerate(flat_shapes)]
        x = [v.view(sh) for v, sh in zip(x, shp)]
        mom = [[torch.zeros(sh, device=dev) for sh in shp] for _ in range(W)]
        pay = [torch.zeros(tr.payload_bytes, dtype=torch.uint8, device=dev) for _ in range(W)]
        for step in range(2):
            for w in range(W):
                g = [inputs.random_tensor(sh, 100 * step + 10 * w + t, 1e-3, torch.bfloat16, dev).view(shn)
                     for t, (sh, shn) in enumerate(zip(flat_shapes, shp))]
                tr.compress(w, g, mom[w], pay[w])
            tr.decode_apply(pay, x)
        assert tr.device_status() == 0
        out.append((pay, mom, x))
    for w in range(W):
        assert torch.equal(out[0][0][w], out[1][0][w])
        assert all(torch.equal(p.reshape(-1), q.reshape(-1)) for p, q in zip(out[0][1][w], out[1][1][w]))
    assert all(torch.equal(p.reshape(-1), q.reshape(-1)) for p, q in zip(out[0][2], out[1][2]))
    b.set_basis(torch.eye(s))
    a.close()
    b.close()


def test_argument_errors_and_unsupported_calls():
    kw = dict(topk=4, beta=0.9, lr=1e-3, weight_decay=0.0, num_workers=1)
    for shapes, chunks, status in (
            ([(10, 10)], [(3, 5)], 2),            # 10 is not a multiple of 3
            ([(8, 8, 8, 8, 8)], [(2,) * 5], 2),   # order 5
            ([(256, 8)], [(256, 1)], 4),          # extent above 128
            ([(128, 128, 2)], [(128, 128, 2)], 4),  # chunk above 16384 elements
            ([(8, 8)], [(0, 8)], 2)):
        with pytest.raises(demo.DemoError) as ei:
            demo.DemoTransform(shapes, chunk_shapes=chunks, **kw)
        assert ei.value.status == status, (shapes, chunks)
    with pytest.raises(demo.DemoError) as ei:
        demo.DemoTransform([(8, 8)], chunk_shapes=[(4, 4)], **dict(kw, topk=0))
    assert ei.value.status == 3
    tr = demo.DemoTransform([(8, 8)], chunk_shapes=[(4, 2)], **kw)
    eye = torch.eye(4)
    assert tr.lib.demo_set_basis(tr._ctx, eye.data_ptr(), None) == 4      # one basis per extent: DCT only
    assert tr.lib.demo_set_basis_gaussian(tr._ctx, eye.data_ptr(), None) == 4
    assert tr.lib.demo_get_basis(tr._ctx, eye.data_ptr(), None) == 4
    tr.close()


def test_randomized_configurations():
    """Seeded random orders, shapes, chunk shapes, k, W, dtypes and decode modes.  Gradients stay at
    1e-3 .. 1e-2: with O(1) data and k close to M the residual is a few fp32 ulp of the chunk, which the
    absolute tolerance of 1e-7 does not cover (the arithmetic, not the kernel, sets that limit)."""
    rng = np.random.default_rng(2024)
    for case in range(16):
        T = int(rng.integers(1, 4))
        shapes, chunks = [], []
        for _ in range(T):
            d = int(rng.integers(1, 5))
            while True:
                ch = tuple(int(rng.choice([1, 2, 3, 4, 5, 8, 12, 16, 32])) for _ in range(d))
                if np.prod(ch) <= 4096:
                    break
            grid = tuple(int(rng.integers(1, 4)) for _ in range(d))
            shapes.append(tuple(c * g for c, g in zip(ch, grid)))
            chunks.append(ch)
        k = int(rng.choice([1, 2, 5, 16, 33]))
        r = parity.NdRunner(shapes, chunks, topk=k, num_workers=int(rng.integers(1, 4)),
                            grad_dtype=torch.float32 if rng.random() < 0.5 else torch.bfloat16,
                            grad_std=float(rng.choice([1e-3, 1e-2])), seed=case,
                            alpha=float(rng.choice([1.0, 0.5])), agg=int(rng.integers(0, 3)), phi=int(rng.integers(0, 2)))
        for _ in range(2):
            r.step()
        r.close()


def test_dimensions_that_are_not_multiples_of_the_target_chunk():
    """A vocabulary-sized matrix (50257 = 29 * 1733 rows) and a 7 x 7 convolution weight: every axis gets
    the largest divisor below the target, and the step matches the oracle on every chunk."""
    from paper_2411_19870_b200 import chunking

    shapes = [(29 * 6, 192), (16, 24, 7, 7), (1000,)]
    chunks = [chunking.divisor_chunk_shape(s, 64) for s in shapes]
    assert chunks == [(58, 64), (16, 12, 7, 7), (50,)]  # 16*24*49 elements would be too many
    r = parity.NdRunner(shapes, chunks, topk=32, num_workers=2)
    for _ in range(2):
        r.step()
    r.close()
