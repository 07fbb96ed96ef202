"""Parameter-server form of the server side (Algorithm 1: the server hands out the sign of the
reconstructed momentum, the workers apply it): demo_decode_signs + demo_apply_signs against
demo_decode_apply and against the oracle's decode."""
import numpy as np
import pytest
import torch

import paper_2411_19870_b200 as demo
from paper_2411_19870_b200 import inputs
from tests import parity

pytestmark = pytest.mark.gpu


def _compress_all(r):
    for w in range(r.wl.num_workers):
        r.tr.compress(w, r.streams[w].next(), r.mom[w], r.payloads[w])


def _server_step(r):
    """One step in both forms from the same payloads and parameters: (x_direct, x_server, signs, x_before)."""
    _compress_all(r)
    x0 = [x.clone() for x in r.params]
    xa = [x.clone() for x in x0]
    xb = [x.clone() for x in x0]
    signs = [torch.full(x.shape, 77, dtype=torch.int8, device=x.device) for x in x0]
    r.tr.decode_apply(r.payloads, xa)
    r.tr.decode_signs(r.payloads, signs)
    r.tr.apply_signs(signs, xb)
    assert r.tr.device_status() == 0
    return xa, xb, signs, x0


@pytest.mark.parametrize("name,path", [("tiny", None), ("small_s64", demo.DEMO_PATH_AUTO), ("small_s64", demo.DEMO_PATH_GENERIC),
                                       ("small_s32", demo.DEMO_PATH_AUTO), ("small_s128", demo.DEMO_PATH_AUTO)])
def test_signs_then_apply_equals_decode_apply_and_the_oracle(name, path):
    wl = inputs.tiny() if name == "tiny" else inputs.small_decoder(chunk=int(name.split("_s")[1]), num_workers=3)
    r = parity.Runner(wl, max_chunks=10**9, path=path)
    r.step()  # an ordinary step first, so that the momenta are not zero
    xa, xb, signs, x0 = _server_step(r)
    s = wl.chunk
    for t, shp in enumerate(wl.shapes):
        sg = signs[t]
        assert sg.dtype == torch.int8 and int(sg.abs().max()) <= 1  # every element was written, values in {-1, 0, 1}
        dense_kernels = path == demo.DEMO_PATH_GENERIC or len(shp) == 1 or s in (8, 16)
        if dense_kernels:
            assert torch.equal(xa[t], xb[t]), "tensor %d: the two forms differ on the dense kernels" % t
        else:  # the fast kernels fold (1 - lr wd) into one factor: one rounding apart
            assert torch.allclose(xa[t], xb[t], rtol=3e-7, atol=1e-9)
        # against the oracle, fed the GPU-written payload bytes (sign exemption band as for demo_decode_apply)
        rows = s if len(shp) == 2 else 1
        first, n_chunks, k_eff = r.layout[t]
        ids = np.arange(n_chunks, dtype=np.int64)
        recs = np.stack([parity.gather_records(r.payloads[w], first, k_eff, ids) for w in range(wl.num_workers)])
        parity.check_decode_chunks(recs, parity.gather_tiles(x0[t], s, ids), parity.gather_tiles(xb[t], s, ids), s, rows,
                                   r.lr, r.wd, r.report, what="server form t%d" % t)
        # the int8 tensor itself: sign of the oracle's R outside the exemption band
        R = parity.orc.decode_chunks(recs, parity.gather_tiles(x0[t], s, ids), s, rows, r.lr, r.wd)["R"]
        got = parity.gather_tiles(sg.to(torch.float32), s, ids)
        exempt = np.abs(R) < parity.SIGN_EXEMPT * np.maximum(1.0, np.max(np.abs(R), axis=1, keepdims=True))
        assert np.all((got == np.sign(R)) | exempt)
    r.close()


@pytest.mark.parametrize("agg", [1, 2])
def test_aggregation_variants_and_refusal_of_the_identity_update(agg):
    wl = inputs.small_decoder(num_workers=4)
    r = parity.Runner(wl, max_chunks=10**9, agg=agg, phi=0)
    xa, xb, _, _ = _server_step(r)
    for a, b in zip(xa, xb):
        assert torch.allclose(a, b, rtol=3e-7, atol=1e-9)
    r.tr.set_decode_mode(agg, demo.DEMO_PHI_IDENTITY)
    signs = [torch.zeros(x.shape, dtype=torch.int8, device=x.device) for x in r.params]
    with pytest.raises(demo.DemoError) as ei:
        r.tr.decode_signs(r.payloads, signs)
    assert ei.value.status == 1
    r.close()


def test_custom_basis_and_rectangular_chunks():
    # caller-supplied basis at s = 64: the signs come from the dense kernels
    wl = inputs.small_decoder(num_workers=2)
    r = parity.Runner(wl, max_chunks=10**9, gauss=inputs.basis_gaussian(11, 64).numpy())
    xa, xb, _, _ = _server_step(r)
    for a, b in zip(xa, xb):
        assert torch.allclose(a, b, rtol=3e-7, atol=1e-9)  # decode_apply ran on the tensor-core kernels
    r.close()
    # tensors of order 3 and 4 with rectangular chunks
    n = parity.NdRunner([(8, 12, 20), (4, 6, 8, 16), (35,)], [(4, 3, 5), (2, 3, 4, 8), (7,)], topk=6, num_workers=2)
    n.step()
    x0 = [x.clone() for x in n.params]
    xa = [x.clone() for x in x0]
    xb = [x.clone() for x in x0]
    signs = [torch.full(x.shape, 77, dtype=torch.int8, device=x.device) for x in x0]
    n.tr.decode_apply(n.payloads, xa)
    n.tr.decode_signs(n.payloads, signs)
    n.tr.apply_signs(signs, xb)
    for a, b, sg in zip(xa, xb, signs):
        assert torch.equal(a, b) and int(sg.abs().max()) <= 1
    n.close()


def test_zero_payloads_give_zero_signs_and_plain_weight_decay():
    wl = inputs.small_decoder(num_workers=2)
    r = parity.Runner(wl, max_chunks=4)
    _compress_all(r)
    for p in r.payloads:
        p.view(torch.float32).view(-1, 2)[:, 1] = 0.0  # every record value 0, indices kept
    x0 = [x.clone() for x in r.params]
    signs = [torch.full(x.shape, 77, dtype=torch.int8, device=x.device) for x in x0]
    r.tr.decode_signs(r.payloads, signs)
    r.tr.apply_signs(signs, r.params)
    for sg, a, b in zip(signs, x0, r.params):
        assert int(sg.abs().max()) == 0
        assert torch.allclose(b, a * (1.0 - r.lr * r.wd), rtol=2e-7, atol=0)  # x (1 - lr wd): plain weight decay
    r.close()


def test_parameter_server_step_in_a_world_of_one():
    """DistributedDemo.step_server through a single-rank NCCL group (gather, decode to signs, broadcast,
    apply): same payload and momentum bits as the direct calls, parameters equal to decode_apply's within the
    rounding of the fast kernels' folded update."""
    import os

    import torch.distributed as dist

    from paper_2411_19870_b200.distributed import DistributedDemo

    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(37500 + (os.getpid() % 2000))
    wl = inputs.small_decoder(num_workers=1)
    r = parity.Runner(wl, max_chunks=8)
    grads = r.streams[0].next()
    dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda", 0))
    try:
        dd = DistributedDemo(wl.shapes, chunk=wl.chunk, topk=wl.topk, beta=wl.beta, lr=wl.lr, weight_decay=wl.weight_decay,
                             grad_dtype=r.tr.cfg.grad_dtype)
        mom = [torch.zeros_like(m) for m in r.mom[0]]
        params = [p.clone() for p in r.params]
        for _ in range(2):
            dd.step_server(grads, mom, params)
        torch.cuda.synchronize()
        assert dd.tr.device_status() == 0
        for _ in range(2):
            r.step(check=True, grads=[grads])
        torch.cuda.synchronize()
        assert all(torch.equal(a, b) for a, b in zip(mom, r.mom[0]))
        assert torch.equal(dd.slices[0], r.payloads[0])
        assert all(torch.allclose(a, b, rtol=6e-7, atol=1e-9) for a, b in zip(params, r.params))
        assert all(int(s.abs().max()) <= 1 for s in dd.signs)
        dd.close()
    finally:
        dist.destroy_process_group()
    r.close()
