"""Out-of-bounds evidence without a memory checker: compress and decode of every kernel family run on
buffers wrapped in guard bands (tests/guards.py); the bands must come back untouched.  The kernels reach
gradients, momentum, parameters and payloads through raw pointers taken from tables, so this is the check
that those tables and the chunk arithmetic stay inside what the caller handed over."""
import numpy as np
import pytest
import torch

import paper_2411_19870_b200 as demo
from paper_2411_19870_b200 import inputs
from tests import parity
from tests.guards import Guarded, all_intact

pytestmark = pytest.mark.gpu

SHAPES = [(256, 384), (128, 256), (128,), (384,)]

# name, chunk, topk, gradient dtype, forced path ("dct": momentum kept in the transform domain), caller-supplied
# basis, chunk shapes (N-D context)
FAMILIES = [
    ("fast_s64_momentum_dct", 64, 32, torch.bfloat16, "dct", False, None),
    ("fast_s64_momentum_dct_k_above_s", 64, 128, torch.float32, "dct", False, None),
    ("fast_s32_bf16", 32, 8, torch.bfloat16, None, False, None),
    ("fast_s32_k_above_s", 32, 100, torch.bfloat16, None, False, None),
    ("fast_s64_bf16", 64, 32, torch.bfloat16, None, False, None),
    ("fast_s64_f32", 64, 32, torch.float32, None, False, None),
    ("fast_s64_k_above_s", 64, 128, torch.bfloat16, None, False, None),
    ("fast_s128_bf16", 128, 32, torch.bfloat16, None, False, None),
    ("generic_s64", 64, 32, torch.bfloat16, "generic", False, None),
    ("generic_s8_f32", 8, 4, torch.float32, None, False, None),
    ("tensor_core_s64", 64, 32, torch.bfloat16, None, True, None),
    ("nd_rectangular", 0, 16, torch.bfloat16, None, False, [(32, 64), (64, 32), (64,), (128,)]),
]


@pytest.mark.parametrize("name,chunk,topk,gdtype,path,custom_basis,chunk_shapes", FAMILIES, ids=[f[0] for f in FAMILIES])
def test_no_kernel_family_writes_outside_its_buffers(name, chunk, topk, gdtype, path, custom_basis, chunk_shapes):
    dev = torch.device("cuda")
    W = 2
    gd = demo.DEMO_BF16 if gdtype == torch.bfloat16 else demo.DEMO_F32
    tr = demo.DemoTransform(SHAPES, chunk=chunk, topk=topk, beta=0.999, lr=1e-3, weight_decay=0.1, num_workers=W,
                            grad_dtype=gd, chunk_shapes=chunk_shapes)
    if path == "generic":
        tr.set_path(demo.DEMO_PATH_GENERIC)
    if path == "dct":
        tr.set_momentum_domain(demo.DEMO_MOMENTUM_DCT)
    if custom_basis:
        q, _ = np.linalg.qr(np.random.default_rng(5).standard_normal((chunk, chunk)))
        tr.set_basis(torch.from_numpy(np.ascontiguousarray(q, dtype=np.float32)))
    gen = torch.Generator(device=dev).manual_seed(77)
    grads = [[Guarded(s, gdtype, dev, fill=(1e-3 * torch.randn(s, generator=gen, device=dev)).to(gdtype)) for s in SHAPES]
             for _ in range(W)]
    mom = [[Guarded(s, torch.float32, dev) for s in SHAPES] for _ in range(W)]
    params = [Guarded(s, torch.float32, dev, fill=0.02 * torch.randn(s, generator=gen, device=dev)) for s in SHAPES]
    payloads = [Guarded((tr.payload_bytes,), torch.uint8, dev) for _ in range(W)]
    x0 = [p.t.clone() for p in params]
    for step in range(2):
        for w in range(W):
            tr.compress(w, [g.t for g in grads[w]], [m.t for m in mom[w]], payloads[w].t)
        tr.decode_apply([p.t for p in payloads], [p.t for p in params])
    torch.cuda.synchronize()
    assert tr.device_status() == 0
    assert all(not torch.equal(p.t, x) for p, x in zip(params, x0))       # the step did run
    assert all(bool((m.t != 0).any().item()) for mw in mom for m in mw)
    everything = [g for gw in grads for g in gw] + [m for mw in mom for m in mw] + params + payloads
    assert all_intact(everything), name + ": a guard band was written"
    tr.close()


def test_parameter_server_form_keeps_inside_its_buffers():
    dev = torch.device("cuda")
    tr = demo.DemoTransform(SHAPES, chunk=64, topk=32, beta=0.999, lr=1e-3, weight_decay=0.1, num_workers=1)
    gen = torch.Generator(device=dev).manual_seed(78)
    g = [(1e-3 * torch.randn(s, generator=gen, device=dev)).bfloat16() for s in SHAPES]
    m = [torch.zeros(s, device=dev) for s in SHAPES]
    payload = Guarded((tr.payload_bytes,), torch.uint8, dev)
    signs = [Guarded(s, torch.int8, dev) for s in SHAPES]
    params = [Guarded(s, torch.float32, dev, fill=0.02 * torch.randn(s, generator=gen, device=dev)) for s in SHAPES]
    tr.compress(0, g, m, payload.t)
    tr.decode_signs([payload.t], [s.t for s in signs])
    tr.apply_signs([s.t for s in signs], [p.t for p in params])
    torch.cuda.synchronize()
    assert tr.device_status() == 0
    assert all_intact([payload] + signs + params)
    tr.close()


@pytest.mark.parametrize("s", [64, 128])
def test_alternating_buffer_sets_at_one_table_slot(s):
    """The library caches pointer tables and TMA tensor maps per worker slot and rewrites them when the caller's
    pointers change.  Two buffer sets take turns at worker slot 0, every step is compared with the oracle on
    every chunk: a kernel that still used the previous set's descriptor would read or write the wrong set."""
    dev = torch.device("cuda")
    wl = inputs.Workload("alternating", [(256, 256), (128, 384)], chunk=s, topk=16, num_workers=1, grad_kind="normal")
    tr = demo.DemoTransform(wl.shapes, chunk=s, topk=wl.topk, beta=wl.beta, lr=wl.lr, weight_decay=wl.weight_decay,
                            num_workers=1)
    beta, lr, wd = (float(np.float32(v)) for v in (wl.beta, wl.lr, wl.weight_decay))
    sets = []
    for i in range(2):
        stream = inputs.GradStream(wl, 10 + i, dev)
        sets.append(dict(stream=stream, m=inputs.make_momentum(wl, dev), x=inputs.make_params(wl, dev),
                         p=torch.zeros(tr.payload_bytes, dtype=torch.uint8, device=dev)))
    rep = parity.Report()
    layout = [tr.payload_layout(t) for t in range(len(wl.shapes))]
    for step in range(6):
        cur = sets[step % 2]
        other = sets[1 - step % 2]
        g = cur["stream"].next()
        ids = [np.arange(layout[t][1], dtype=np.int64) for t in range(len(wl.shapes))]
        before = [parity.gather_tiles(cur["m"][t], s, ids[t]) for t in range(len(wl.shapes))]
        other_m = [m.clone() for m in other["m"]]
        other_x = [x.clone() for x in other["x"]]
        tr.compress(0, g, cur["m"], cur["p"])
        for t in range(len(wl.shapes)):
            parity.check_compress_chunks(parity.gather_tiles(g[t], s, ids[t]), before[t],
                                         parity.gather_tiles(cur["m"][t], s, ids[t]),
                                         parity.gather_records(cur["p"], layout[t][0], layout[t][2], ids[t]), s, s,
                                         wl.topk, beta, rep, what="step %d t%d" % (step, t))
        xb = [parity.gather_tiles(cur["x"][t], s, ids[t]) for t in range(len(wl.shapes))]
        tr.decode_apply([cur["p"]], cur["x"])
        for t in range(len(wl.shapes)):
            recs = parity.gather_records(cur["p"], layout[t][0], layout[t][2], ids[t])[None]
            parity.check_decode_chunks(recs, xb[t], parity.gather_tiles(cur["x"][t], s, ids[t]), s, s, lr, wd, rep,
                                       what="decode step %d t%d" % (step, t))
        # the set that is not in use stays as it was
        assert all(torch.equal(a, b) for a, b in zip(other_m, other["m"]))
        assert all(torch.equal(a, b) for a, b in zip(other_x, other["x"]))
    assert tr.device_status() == 0
    tr.close()
