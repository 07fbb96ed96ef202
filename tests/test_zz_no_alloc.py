"""demo_decode_apply_static: the decode + update entry point for callers that may not allocate
(memory-pool owners, plug-ins barred from driver allocations after start-up).  Its tables live in a
fixed device array instead of cudaMalloc'ed memory, so the risks it carries are stale or misplaced
table contents and an allocation slipping in -- checked here by calling it several times in a row with
different tensor sets, chunk sizes, payloads and parameters, against the context-based entry point and
against the fp64 oracle, with the device's free memory compared across the calls.  Collected last on
purpose: a failure here cannot hide another test's result in a run that stops at the first failure."""
import numpy as np
import pytest
import torch

import paper_2411_19870_b200 as demo
from paper_2411_19870_b200 import inputs
from tests import parity

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


def _check_against_oracle(wl, tr, payloads, before, after, max_chunks=48):
    """Sampled chunks of every tensor: the parameters the static call left against the oracle's decode of the
    same payload bytes (the rule of every other parity test)."""
    rep = parity.Report()
    s = wl.chunk
    for t, shp in enumerate(wl.shapes):
        first, n_chunks, k_eff = tr.payload_layout(t)
        ids = parity.sample_chunk_ids(n_chunks, max_chunks, 100 + t)
        rows = s if len(shp) == 2 else 1
        recs = np.stack([parity.gather_records(p, first, k_eff, ids) for p in payloads])
        parity.check_decode_chunks(recs, parity.gather_tiles(before[t], s, ids), parity.gather_tiles(after[t], s, ids),
                                   s, rows, float(np.float32(wl.lr)), float(np.float32(wl.weight_decay)), rep,
                                   what="static decode t%d" % t)
    assert rep["decode_chunks"] > 0
    return rep


def test_static_entry_point_matches_context_entry_point_and_oracle_on_changing_shapes():
    # Four calls in a row through the one shared table array: a mixed 2-D / 1-D set at s = 64, the same set again
    # with other payloads and parameter buffers, a smaller set at s = 32 (fewer tensors, other basis: anything
    # left over from the earlier, larger calls would show), and a set of 1-D tensors only.
    cases = [
        inputs.small_decoder(num_workers=3),
        inputs.small_decoder(num_workers=3),
        inputs.Workload("two_matrices_s32", [(128, 96), (64, 64), (96,)], chunk=32, topk=5, num_workers=2,
                        grad_kind="normal"),
        inputs.Workload("vectors_only", [(256,), (64,)], chunk=64, topk=9, num_workers=2, grad_kind="normal"),
    ]
    free_after_first = None
    for call, wl in enumerate(cases):
        kw = dict(chunk=wl.chunk, topk=wl.topk, lr=wl.lr, weight_decay=wl.weight_decay)
        tr, payloads, params = _payloads_and_params(wl, steps=1 + call % 2)
        ref_generic = [p.clone() for p in params]
        ref_fast = [p.clone() for p in params]
        got = [p.clone() for p in params]
        tr.set_path(demo.DEMO_PATH_GENERIC)
        tr.decode_apply(payloads, ref_generic)
        tr.set_path(demo.DEMO_PATH_AUTO)
        tr.decode_apply(payloads, ref_fast)
        torch.cuda.synchronize()
        # the library must not allocate: free device memory (driver's view, below torch's caching allocator)
        # is the same before and after the call; the first call of the process is let through once because
        # the driver may load the kernels' module lazily on first use
        free_before = torch.cuda.mem_get_info()[0]
        demo.decode_apply_static(wl.shapes, payloads, got, **kw)
        torch.cuda.synchronize()
        free_after = torch.cuda.mem_get_info()[0]
        if call > 0:
            assert free_after == free_before, "device memory changed across demo_decode_apply_static"
        assert tr.device_status() == 0
        for g, rg, rf, p0 in zip(got, ref_generic, ref_fast, params):
            assert not torch.equal(g, p0)          # it did update
            assert torch.equal(g, rg)              # same kernels as the generic path: bit-identical
            # against the fast path: the tolerance of the parity tests, sign flips only at |R| ~ 0
            close = torch.isclose(g, rf, rtol=1e-5, atol=1e-7)
            assert close.float().mean().item() > 0.9999
        _check_against_oracle(wl, tr, payloads, params, got)
        tr.close()


def test_static_entry_point_skips_a_record_outside_its_chunk():
    # One record of one worker gets an index beyond the chunk: the entry point must leave the parameters the
    # oracle computes from the payload WITHOUT that record (it has no context through which to report it).
    wl = inputs.Workload("one_matrix", [(128, 128)], chunk=64, topk=8, num_workers=2, grad_kind="normal")
    tr, payloads, params = _payloads_and_params(wl, steps=1)
    first, n_chunks, k_eff = tr.payload_layout(0)
    rec = payloads[1].view(torch.int32).view(-1, 2)
    victim = first + 2 * k_eff + 3          # chunk 2, record 3 of worker 1
    rec[victim, 0] = 64 * 64 + 17           # outside the chunk
    got = [p.clone() for p in params]
    demo.decode_apply_static(wl.shapes, payloads, got, chunk=wl.chunk, topk=wl.topk, lr=wl.lr,
                             weight_decay=wl.weight_decay)
    torch.cuda.synchronize()
    ids = np.arange(n_chunks, dtype=np.int64)
    recs = np.stack([parity.gather_records(p, first, k_eff, ids) for p in payloads])
    recs[1, 2, 3] = (0, 0.0)                # the oracle sees the record dropped: index 0 with value 0 adds nothing
    rep = parity.Report()
    parity.check_decode_chunks(recs, parity.gather_tiles(params[0], 64, ids), parity.gather_tiles(got[0], 64, ids), 64, 64,
                               float(np.float32(wl.lr)), float(np.float32(wl.weight_decay)), rep, what="dropped record")
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


def test_static_entry_point_refuses_a_capturing_stream():
    # its table copies read host memory that is gone after the call: they must not end up in a graph
    dev = torch.device("cuda")
    wl = inputs.Workload("one_matrix", [(64, 64)], chunk=64, topk=4, num_workers=1, grad_kind="normal")
    tr, payloads, params = _payloads_and_params(wl, steps=1)
    kw = dict(chunk=wl.chunk, topk=wl.topk, lr=wl.lr, weight_decay=wl.weight_decay)
    demo.decode_apply_static(wl.shapes, payloads, [p.clone() for p in params], **kw)  # set-up outside any capture
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    untouched = [p.clone() for p in params]
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        graph.capture_begin()
        try:
            with pytest.raises(demo.DemoError) as e:
                demo.decode_apply_static(wl.shapes, payloads, untouched, stream=side, **kw)
            assert e.value.status == 1
        finally:
            graph.capture_end()
    torch.cuda.synchronize()
    assert all(torch.equal(a, b) for a, b in zip(untouched, params))  # nothing was enqueued
    tr.close()
