"""demo_decode_apply_static: the decode + update entry point for callers that may not allocate
(memory-pool owners, plug-ins barred from driver allocations after start-up).  Its tables live in a
fixed device array instead of cudaMalloc'ed memory, so the risk it carries is stale or misplaced
table contents -- checked here by running it twice in a row, on different payloads and parameters,
against the context-based entry point.  Collected last on purpose: a failure here cannot hide
another test's result in a run that stops at the first failure."""
import pytest
import torch

import paper_2411_19870_b200 as demo
from paper_2411_19870_b200 import inputs

pytestmark = pytest.mark.gpu


def _payloads_and_params(wl, steps):
    """Run `steps` compress rounds through a context; return the transform, payloads and fresh params."""
    dev = torch.device("cuda")
    tr = demo.DemoTransform(wl.shapes, chunk=wl.chunk, topk=wl.topk, beta=wl.beta, lr=wl.lr,
                            weight_decay=wl.weight_decay, num_workers=wl.num_workers)
    mom = [inputs.make_momentum(wl, dev) for _ in range(wl.num_workers)]
    streams = [inputs.GradStream(wl, w, dev) for w in range(wl.num_workers)]
    payloads = [torch.zeros(tr.payload_bytes, dtype=torch.uint8, device=dev) for _ in range(wl.num_workers)]
    for _ in range(steps):
        for w in range(wl.num_workers):
            tr.compress(w, streams[w].next(), mom[w], payloads[w])
    return tr, payloads, inputs.make_params(wl, dev)


def test_static_entry_point_matches_context_entry_point_twice():
    wl = inputs.small_decoder(num_workers=3)  # 2-D and 1-D tensors, s=64, k=32
    kw = dict(chunk=wl.chunk, topk=wl.topk, lr=wl.lr, weight_decay=wl.weight_decay)
    for call in range(2):  # second call: other payloads, other parameter buffers, same shared tables
        tr, payloads, params = _payloads_and_params(wl, steps=1 + call)
        ref_generic = [p.clone() for p in params]
        ref_fast = [p.clone() for p in params]
        got = [p.clone() for p in params]
        tr.set_path(demo.DEMO_PATH_GENERIC)
        tr.decode_apply(payloads, ref_generic)
        tr.set_path(demo.DEMO_PATH_AUTO)
        tr.decode_apply(payloads, ref_fast)
        demo.decode_apply_static(wl.shapes, payloads, got, **kw)
        torch.cuda.synchronize()
        assert tr.device_status() == 0
        for g, rg, rf, p0 in zip(got, ref_generic, ref_fast, params):
            assert not torch.equal(g, p0)          # it did update
            assert torch.equal(g, rg)              # same kernels as the generic path: bit-identical
            # against the fast path: the tolerance of the parity tests, sign flips only at |R| ~ 0
            close = torch.isclose(g, rf, rtol=1e-5, atol=1e-7)
            assert close.float().mean().item() > 0.9999
        tr.close()


def test_static_entry_point_rejects_what_does_not_fit():
    dev = torch.device("cuda")
    x = [torch.zeros(128, 128, device=dev)]
    p = [torch.zeros(4 * 8 * 8, dtype=torch.uint8, device=dev)]
    with pytest.raises(demo.DemoError) as e:   # chunk size beyond the fixed basis table
        demo.decode_apply_static([(128, 128)], p, x, chunk=128, topk=8, lr=1e-3, weight_decay=0.0)
    assert e.value.status == 4
    many = [(64, 64)] * 257                     # more tensors than the fixed tensor table holds
    with pytest.raises(demo.DemoError) as e:
        demo.decode_apply_static(many, p, x * 257, chunk=64, topk=8, lr=1e-3, weight_decay=0.0)
    assert e.value.status == 4
    with pytest.raises(demo.DemoError) as e:   # more payloads than the fixed pointer table holds
        demo.decode_apply_static([(128, 128)], p * 65, x, chunk=64, topk=8, lr=1e-3, weight_decay=0.0)
    assert e.value.status == 4
