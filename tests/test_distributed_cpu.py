"""One worker per rank (the exchange of Section 2.1): the host side -- slice layout of the gather
buffer, rank order = worker order, every rank ending with the same parameters -- with two gloo ranks
on CPU.  The compress and decode kernels need a GPU, so the oracle stands in for them here; the GPU
suite runs the real kernels through the same class in a world of one."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

S, K, BETA, LR, WD = 8, 4, 0.9, 1e-3, 0.1
SHAPES = [(16, 24), (32,)]


def _inputs(rank):
    rng = np.random.default_rng(100 + rank)
    g = [rng.standard_normal(s).astype(np.float32) for s in SHAPES]
    m = [rng.standard_normal(s).astype(np.float32) * 0.1 for s in SHAPES]
    return g, m


def _params():
    rng = np.random.default_rng(7)
    return [rng.standard_normal(s).astype(np.float32) * 0.02 for s in SHAPES]


def _payload_bytes(orc, g, m):
    """This worker's payload: tensors concatenated in order, chunk-major records."""
    parts = [orc.compress_tensor(gt, mt, S, K, BETA)["records"].reshape(-1) for gt, mt in zip(g, m)]
    return np.concatenate(parts).view(np.uint8)


def _decode(orc, slices, x):
    """Oracle decode of the gathered slices (worker order = slice order)."""
    out, first = [], 0
    for xt in x:
        n_chunks = xt.size // (S * S if xt.ndim == 2 else S)
        k_eff = min(K, S * S if xt.ndim == 2 else S)
        n = n_chunks * k_eff
        recs = [sl.view(orc.RECORD_DTYPE)[first:first + n].reshape(n_chunks, k_eff) for sl in slices]
        out.append(orc.decode_tensor(recs, xt, S, K, LR, WD)["x_new"])
        first += n
    return out


def _rank_main(rank, world, port, out):
    from oracle import demo_oracle as orc
    from paper_2411_19870_b200.distributed import gather_payloads

    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    g, m = _inputs(rank)
    mine = _payload_bytes(orc, g, m)
    pb = mine.size
    buffer = torch.zeros(world * pb, dtype=torch.uint8)
    slices = [buffer[w * pb:(w + 1) * pb] for w in range(world)]
    slices[rank].copy_(torch.from_numpy(mine.copy()))
    gather_payloads(slices, buffer, rank)
    x_new = _decode(orc, [s.numpy() for s in slices], _params())
    out.put((rank, buffer.numpy().tobytes(), [x.tobytes() for x in x_new]))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_gather_in_worker_order_and_agree():
    from oracle import demo_oracle as orc

    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 31500 + (os.getpid() % 2000)
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = dict()
    for _ in range(2):
        rank, buf, xs = out.get(timeout=120)
        got[rank] = (buf, xs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    # both ranks hold the same gathered bytes and the same parameters afterwards
    assert got[0][0] == got[1][0] and got[0][1] == got[1][1]
    # slice w is worker w's payload, and the update is the single-process two-worker step
    want = [_payload_bytes(orc, *_inputs(w)) for w in range(2)]
    assert got[0][0] == b"".join(w.tobytes() for w in want)
    ref = _decode(orc, want, _params())
    assert [x.tobytes() for x in ref] == got[0][1]


def _server_rank_main(rank, world, port, out):
    """Parameter-server form on two gloo ranks: gather on rank 1, oracle decode there, int8 signs broadcast."""
    from oracle import demo_oracle as orc
    from paper_2411_19870_b200.distributed import broadcast_signs, gather_to_server, sign_views

    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    server = 1
    g, m = _inputs(rank)
    mine = _payload_bytes(orc, g, m)
    pb = mine.size
    buffer = torch.zeros(world * pb, dtype=torch.uint8)
    slices = [buffer[w * pb:(w + 1) * pb] for w in range(world)]
    slices[rank].copy_(torch.from_numpy(mine.copy()))
    gather_to_server(slices, rank, server)
    flat, views = sign_views(SHAPES, "cpu")
    assert all(v.data_ptr() % 16 == 0 for v in views) and [tuple(v.shape) for v in views] == SHAPES
    x = _params()
    if rank == server:
        first = 0
        for xt, v in zip(x, views):
            n_chunks = xt.size // (S * S if xt.ndim == 2 else S)
            k_eff = min(K, S * S if xt.ndim == 2 else S)
            n = n_chunks * k_eff
            recs = [sl.numpy().view(orc.RECORD_DTYPE)[first:first + n].reshape(n_chunks, k_eff) for sl in slices]
            R = orc.decode_tensor(recs, xt, S, K, LR, WD)["R"]
            v.copy_(torch.from_numpy(np.sign(R).astype(np.int8)))
            first += n
    broadcast_signs(flat, server)
    x_new = [xt.astype(np.float64) - LR * (v.numpy().astype(np.float64) + WD * xt.astype(np.float64)) for xt, v in zip(x, views)]
    out.put((rank, flat.numpy().tobytes(), [a.tobytes() for a in x_new]))
    dist.barrier()
    dist.destroy_process_group()


def test_parameter_server_form_on_two_gloo_ranks():
    from oracle import demo_oracle as orc

    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 35500 + (os.getpid() % 2000)
    procs = [ctx.Process(target=_server_rank_main, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = dict()
    for _ in range(2):
        rank, signs, xs = out.get(timeout=120)
        got[rank] = (signs, xs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    # both ranks received the server's signs and end with the parameters of the all-gather form
    assert got[0] == got[1]
    want = [_payload_bytes(orc, *_inputs(w)) for w in range(2)]
    ref = _decode(orc, want, _params())
    for a, b in zip(ref, got[0][1]):
        np.testing.assert_allclose(np.frombuffer(b, dtype=np.float64), np.asarray(a, dtype=np.float64).reshape(-1), rtol=0, atol=1e-15)


def test_gather_rejects_a_buffer_of_the_wrong_size():
    import pytest
    from paper_2411_19870_b200.distributed import gather_payloads

    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(33500 + (os.getpid() % 2000))
    dist.init_process_group("gloo", rank=0, world_size=1)
    try:
        buf = torch.zeros(16, dtype=torch.uint8)
        with pytest.raises(ValueError):
            gather_payloads([buf[:8], buf[8:]], buf, 0)
        gather_payloads([buf], buf, 0)  # a world of one: the slice is the buffer
    finally:
        dist.destroy_process_group()
