"""The five configurations at their full sizes, in the launch configuration the benchmark times, at the
sampling density stated for them: config 2 over all ten steps (every chunk on one step, one chunk in sixteen
on the others, step-locked: the oracle starts every step from the device's previous momentum and parameters);
configs 3, 4 and the full-set half of config 5 with the first, the last and at least one in 64 chunks of every
2-D tensor and every chunk of the 1-D tensors, plus the whole-tensor invariants (every chunk, every worker);
config 5's decode fan-in of 64 workers on the 1B-class set through one scratch momentum buffer."""
import numpy as np
import pytest
import torch

import paper_2411_19870_b200 as demo
from paper_2411_19870_b200 import inputs
from tests import parity
from tests.guards import Guarded, all_intact

pytestmark = pytest.mark.gpu


def _free_gb():
    free, _ = torch.cuda.mem_get_info()
    return free / 1e9


def _one_in_64(runner, seed):
    """first + last + >= 1/64 of the chunks of every tensor; tensors of up to 32 chunks (all 1-D tensors of the
    configured sets) in full"""
    return [parity.sample_chunk_fraction(runner.layout[t][1], 64, seed + t, min_n=32 if len(shp) == 1 else 8)
            for t, shp in enumerate(runner.wl.shapes)]


def test_config2_single_matrix_all_ten_steps_step_locked():
    wl = inputs.single_matrix()
    r = parity.Runner(wl, max_chunks=8)
    n_chunks = r.layout[0][1]
    assert n_chunks == 16384
    for step in range(wl.steps):
        if step == 4:
            r.ids = [np.arange(n_chunks, dtype=np.int64)]       # every chunk, with a momentum that has filled up
        else:
            r.ids = [parity.sample_chunk_fraction(n_chunks, 16, 1000 + step)]
        r.step(invariants=True)
    assert wl.steps == 10
    assert r.report["chunks"] == 16384 + 9 * 1024
    assert r.report["decode_chunks"] == 16384 + 9 * 1024
    assert r.report["invariant_records"] == 10 * wl.records_per_worker()
    r.close()
    torch.cuda.empty_cache()


def test_config3_decoder_300m_one_chunk_in_64_and_invariants():
    wl = inputs.decoder_300m()
    if _free_gb() < 30:
        pytest.skip("not enough free device memory")
    r = parity.Runner(wl, max_chunks=8)
    r.ids = _one_in_64(r, 300)
    per_worker = sum(len(i) for i in r.ids)
    assert per_worker >= 110880 // 64 + 768          # >= 1/64 of the 2-D tiles and all 768 1-D segments
    r.step(invariants=True)
    r.step(invariants=True)
    assert r.report["chunks"] == 2 * wl.num_workers * per_worker
    assert r.report["invariant_records"] == 2 * wl.num_workers * wl.records_per_worker()
    r.close()
    torch.cuda.empty_cache()


def test_config4_decoder_1b_one_chunk_in_64_on_three_workers_and_invariants_on_all():
    wl = inputs.decoder_1b()
    if _free_gb() < 140:
        pytest.skip("not enough free device memory")
    r = parity.Runner(wl, max_chunks=8)
    r.ids = _one_in_64(r, 400)
    per_worker = sum(len(i) for i in r.ids)
    assert per_worker >= 312448 // 64 + 1024
    r.step(workers=(0, 7, 15), invariants=True)
    assert r.report["chunks"] == 3 * per_worker
    assert r.report["decode_chunks"] == per_worker
    assert r.report["invariant_records"] == wl.num_workers * wl.records_per_worker()
    r.close()
    torch.cuda.empty_cache()


def test_config5_stress_full_set_heavy_tails_and_tie_makers():
    wl = inputs.stress(chunk=64, topk=32, num_workers=8, full_set=True)
    if _free_gb() < 80:
        pytest.skip("not enough free device memory")
    r = parity.Runner(wl, max_chunks=8)
    r.ids = _one_in_64(r, 500)
    per_worker = sum(len(i) for i in r.ids)
    r.step(workers=(0, 3, 7), invariants=True)
    assert r.report["chunks"] == 3 * per_worker
    assert r.report["unpinned"] > 0                  # the tie-maker chunks are in the sample
    r.close()
    torch.cuda.empty_cache()


def test_config5_decode_fan_in_of_64_workers_on_the_1b_class_set():
    """One step from zero momentum (m = g): every worker's gradients go through ONE scratch momentum buffer into
    that worker's own payload (64 momenta of the 1B-class set would not fit the device), the residuals are
    discarded, and the decode of the 64 payloads is compared with the oracle.  Payloads, scratch momentum and
    parameters sit in guard bands."""
    wl = inputs.stress(chunk=64, topk=32, num_workers=64, full_set=True)
    if _free_gb() < 40:
        pytest.skip("not enough free device memory")
    dev = torch.device("cuda")
    s, W, T = wl.chunk, wl.num_workers, len(wl.shapes)
    tr = demo.DemoTransform(wl.shapes, chunk=s, topk=wl.topk, beta=wl.beta, lr=wl.lr, weight_decay=wl.weight_decay,
                            num_workers=W)
    beta, lr, wd = (float(np.float32(v)) for v in (wl.beta, wl.lr, wl.weight_decay))
    layout = [tr.payload_layout(t) for t in range(T)]
    ids = [parity.sample_chunk_fraction(layout[t][1], 128, 600 + t, min_n=32 if len(shp) == 1 else 4)
           for t, shp in enumerate(wl.shapes)]
    scratch = [Guarded(shp, torch.float32, dev) for shp in wl.shapes]
    params = [Guarded(shp, torch.float32, dev, fill=p) for shp, p in zip(wl.shapes, inputs.make_params(wl, dev))]
    payloads = [Guarded((tr.payload_bytes,), torch.uint8, dev) for _ in range(W)]
    rep = parity.Report()
    for w in range(W):
        g = inputs.GradStream(wl, w, dev).next()
        for m in scratch:
            m.t.zero_()
        checked = w in (0, 21, 63)
        if checked:
            energy = [parity.tensor_energy(beta, scratch[t].t, g[t]) for t in range(T)]
        tr.compress(w, g, [m.t for m in scratch], payloads[w].t)
        if checked:
            mom = [m.t for m in scratch]
            parity.check_whole_tensor_invariants(payloads[w].t, layout, wl.shapes, s, energy, mom, what="worker %d" % w)
            for t, shp in enumerate(wl.shapes):
                rows = s if len(shp) == 2 else 1
                gt = parity.gather_tiles(g[t], s, ids[t])
                parity.check_compress_chunks(gt, np.zeros_like(gt), parity.gather_tiles(mom[t], s, ids[t]),
                                             parity.gather_records(payloads[w].t, layout[t][0], layout[t][2], ids[t]),
                                             s, rows, wl.topk, beta, rep, what="fan-in compress w%d t%d" % (w, t))
        del g
    xb = [parity.gather_tiles(params[t].t, s, ids[t]) for t in range(T)]
    tr.decode_apply([p.t for p in payloads], [p.t for p in params])
    torch.cuda.synchronize()
    for t, shp in enumerate(wl.shapes):
        rows = s if len(shp) == 2 else 1
        recs = np.stack([parity.gather_records(payloads[w].t, layout[t][0], layout[t][2], ids[t]) for w in range(W)])
        parity.check_decode_chunks(recs, xb[t], parity.gather_tiles(params[t].t, s, ids[t]), s, rows, lr, wd, rep,
                                   what="fan-in decode t%d" % t)
    assert tr.device_status() == 0
    assert rep["decode_chunks"] == sum(len(i) for i in ids)
    assert all_intact(scratch + params + payloads)
    tr.close()
    torch.cuda.empty_cache()
