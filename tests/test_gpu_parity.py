"""GPU parity tests: the CUDA path, called through the C ABI, against the fp64 CPU oracle on the
same seeded inputs (rules in tests/parity.py)."""
import numpy as np
import pytest
import torch

import paper_2411_19870_b200 as demo
from paper_2411_19870_b200 import inputs
from tests import parity

pytestmark = pytest.mark.gpu

PATHS = [demo.DEMO_PATH_AUTO, demo.DEMO_PATH_GENERIC]


def test_library_is_the_cuda_build():
    lib = demo.load_library()
    assert lib._name.endswith("libdemo_b200.so")


def test_tiny_three_steps_all_chunks():
    """Config 1: every chunk of both tensors, 3 steps, W=2, step-locked against the oracle."""
    wl = inputs.tiny()
    r = parity.Runner(wl, max_chunks=10**9)
    for _ in range(wl.steps):
        r.step()
    rep = r.report
    assert rep["chunks"] == 3 * 2 * (2048 + 64) and rep["decode_chunks"] == 3 * (2048 + 64)
    r.close()


@pytest.mark.parametrize("path", PATHS)
def test_small_decoder_s64_k32(path):
    """Scaled-down decoder set (2-D and 1-D tensors), s=64, k=32, W=4, 3 steps, all chunks."""
    wl = inputs.small_decoder()
    r = parity.Runner(wl, max_chunks=10**9, path=path)
    for _ in range(3):
        r.step()
    assert r.report["pinned"] > 0.98 * r.report["chunks"]
    r.close()


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("k", [32, 200])
def test_small_decoder_s128(path, k):
    """Chunk size 128 (the paper's second setting): split 128-point transforms on the fast path."""
    wl = inputs.small_decoder(chunk=128, topk=k, num_workers=3)
    r = parity.Runner(wl, max_chunks=40, path=path)
    for _ in range(2):
        r.step()
    assert r.report["pinned"] > 0.95 * r.report["chunks"]
    r.close()


@pytest.mark.parametrize("path", PATHS)
def test_single_matrix_sampled(path):
    """Config 2 at full size (8192 x 8192, row-scaled bf16 grads), 2 steps, 300 sampled chunks."""
    wl = inputs.single_matrix()
    r = parity.Runner(wl, max_chunks=300, path=path)
    r.step()
    r.step()
    r.close()


@pytest.mark.parametrize("s,k", [(8, 64), (32, 1024), (64, 4096), (64, 64), (128, 16384)])
def test_lossless_when_k_covers_the_chunk(s, k):
    """k = M: zero residual momentum and an update of exactly sign(sum_w m_w)."""
    shapes = [(2 * s, 3 * s), (4 * s,)]
    wl = inputs.Workload("lossless", shapes, chunk=s, topk=k, num_workers=3, grad_kind="normal", grad_std=0.01)
    r = parity.Runner(wl, max_chunks=10**9)
    grads = [st.next() for st in r.streams]
    x0 = [p.clone() for p in r.params]
    r.step(grads=grads)
    tot2d = sum(g[0].double() for g in grads)
    if k >= s * s:
        assert max(m[0].abs().max().item() for m in r.mom) < 1e-7
        sg = torch.sign(tot2d)
        big = tot2d.abs() > 1e-6
        step = torch.round((x0[0].double() * (1 - wl.lr * wl.weight_decay) - r.params[0].double()) / wl.lr)
        assert torch.equal(step[big], sg[big])
    assert max(m[1].abs().max().item() for m in r.mom) < 1e-7  # 1-D segments: k_eff = s
    r.close()


@pytest.mark.parametrize("s", [32, 64, 128])
@pytest.mark.parametrize("k", [1, 8, 32, 128])
def test_stress_matrix_ties(s, k):
    """Config 5 on the 4096 x 4096 matrix: heavy-tailed grads, 5% tie-maker chunks, W=8, 2 steps."""
    wl = inputs.stress(chunk=s, topk=k, num_workers=8, full_set=False)
    r = parity.Runner(wl, max_chunks=160 if s < 128 else 48, seed=s + k)
    r.step()
    r.step()
    assert r.report["unpinned"] > 0  # the tie-makers are really there
    r.close()


def _random_case(seed):
    """A seeded random configuration: chunk size, k (from 1 up to lossless), workers, a mix of 2-D and 1-D
    shapes, gradient family, dtype, alpha, aggregation and phi."""
    rng = np.random.default_rng(1000 + seed)
    s = int(rng.choice([8, 16, 32, 64, 64, 128]))
    M = s * s
    k = int(rng.choice([1, 2, 3, 7, s // 2, s - 1, s, s + 1, 2 * s, min(M, 300), M]))
    W = int(rng.integers(1, 6))
    n2 = int(rng.integers(1, 4))
    shapes = [(s * int(rng.integers(1, 4)), s * int(rng.integers(1, 5))) for _ in range(n2)]
    shapes += [(s * int(rng.integers(1, 6)),) for _ in range(int(rng.integers(0, 3)))]
    kind = str(rng.choice(["normal", "row_lognormal", "tensor_scaled", "student_t_ties"]))
    dtype = torch.bfloat16 if rng.random() < 0.6 else torch.float32
    alpha = None if rng.random() < 0.5 else float(rng.choice([0.2, 0.5, 1.0]))
    agg, phi = int(rng.integers(0, 3)), int(rng.integers(0, 2))
    # the heavy-tailed family keeps the scale of the stress configuration (Student-t x 1e-3): with a larger
    # one an outlier of magnitude ~1 in a lossless chunk leaves a residual of one fp32 ulp of 1 (1.19e-7),
    # which no fp32 subtraction of two O(1) numbers can avoid and the flat 1e-7 bound does not allow
    wl = inputs.Workload("random%d" % seed, shapes, chunk=s, topk=k, num_workers=W, grad_kind=kind,
                         grad_std=1e-3 if kind == "student_t_ties" else 0.01, grad_dtype=dtype)
    return wl, alpha, agg, phi


@pytest.mark.parametrize("seed", range(40))
def test_randomized_configurations_match_the_oracle(seed):
    """Every chunk of a small random configuration, two steps, both kernel families."""
    wl, alpha, agg, phi = _random_case(seed)
    for path in PATHS:
        r = parity.Runner(wl, max_chunks=10**9, path=path, seed=seed, alpha=alpha, agg=agg, phi=phi)
        r.step()
        r.step()
        r.close()


def test_all_zero_chunks_emit_lowest_indices():
    """Exactly tied magnitudes: the deterministic tie-break (lowest index) is bit-testable."""
    for s, shapes in [(64, [(128, 128), (128,)]), (8, [(16, 16), (16,)]), (32, [(64, 64)]), (128, [(256, 128)])]:
        for path in PATHS:
            tr = demo.DemoTransform(shapes, chunk=s, topk=5, beta=0.9, lr=1e-3, weight_decay=0.0, num_workers=1,
                                    grad_dtype=demo.DEMO_F32)
            tr.set_path(path)
            g = [torch.zeros(sh, device="cuda") for sh in shapes]
            m = [torch.zeros(sh, device="cuda") for sh in shapes]
            p = torch.full((tr.payload_bytes,), 0xFF, dtype=torch.uint8, device="cuda")
            tr.compress(0, g, m, p)
            rec = p.view(torch.int32).view(-1, 5, 2).cpu()
            assert torch.equal(rec[:, :, 0], torch.arange(5, dtype=torch.int32).expand(rec.shape[0], 5))
            assert torch.all(rec[:, :, 1] == 0)
            tr.close()


@pytest.mark.parametrize("path", PATHS)
def test_constant_tile_ties_pick_lowest_index_among_equals(path):
    """A tile whose coefficients are +-a exactly (B = C^T (+-a) C is not exactly representable, so
    build the tie in the coefficient domain the other way round: an all-equal tile has one nonzero
    coefficient and M-1 exact... near-zeros; the kept set must still be valid)."""
    s = 64
    wl = inputs.Workload("const", [(s, s)], chunk=s, topk=4, num_workers=1, grad_kind="normal", grad_std=0.0)
    r = parity.Runner(wl, max_chunks=10, path=path)
    g = [torch.full((s, s), 0.5, device="cuda", dtype=torch.bfloat16)]
    r.step(grads=[g])
    rec = r.payloads[0].view(torch.int32).view(-1, 2).cpu()
    assert rec[0, 0].item() == 0  # the DC coefficient a*s is kept
    assert abs(rec[0, 1].view(torch.float32).item() - 32.0) < 1e-4
    r.close()


def test_run_to_run_determinism():
    wl = inputs.small_decoder(num_workers=2)
    outs = []
    for _ in range(2):
        r = parity.Runner(wl, max_chunks=4)
        r.step(check=False)
        r.step(check=False)
        torch.cuda.synchronize()
        outs.append(([p.clone() for p in r.payloads], [x.clone() for x in r.params], [m.clone() for m in r.mom[1]]))
        r.close()
    for a, b in zip(outs[0], outs[1]):
        assert all(torch.equal(x, y) for x, y in zip(a, b))


def test_fast_and_generic_paths_agree():
    wl = inputs.small_decoder(num_workers=2)
    res = []
    for path in PATHS:
        r = parity.Runner(wl, max_chunks=4, path=path)
        r.step(check=False)
        torch.cuda.synchronize()
        res.append((r.payloads[0].view(torch.int32).view(-1, 2).clone(), r.mom[0][0].clone(), r.params[0].clone()))
        r.close()
    same_idx = (res[0][0][:, 0] == res[1][0][:, 0]).float().mean().item()
    assert same_idx > 0.999  # index sets may differ only on near-tied chunks
    assert torch.allclose(res[0][1], res[1][1], rtol=1e-4, atol=1e-7)


def test_full_coverage_invariants_medium_set():
    """Whole-tensor properties that hold at any size, checked on every chunk with torch ops:
    ascending in-range indices and the energy identity ||m_new||^2 = ||beta m + g||^2 - sum val^2."""
    wl = inputs.small_decoder(d_model=512, n_layers=2, vocab=4096, num_workers=2)
    r = parity.Runner(wl, max_chunks=8)
    r.step(check=False)
    g = [st.next() for st in r.streams]
    m_before = [[m.clone() for m in mw] for mw in r.mom]
    r.step(check=False, grads=g)
    for w in range(wl.num_workers):
        rec = r.payloads[w].view(torch.int32).view(-1, 2)
        for t, shp in enumerate(wl.shapes):
            first, n_chunks, k_eff = r.layout[t]
            M = wl.chunk ** 2 if len(shp) == 2 else wl.chunk
            rr = rec[first:first + n_chunks * k_eff].view(n_chunks, k_eff, 2)
            idx = rr[:, :, 0]
            assert idx.min().item() >= 0 and idx.max().item() < M
            assert torch.all(idx[:, 1:] > idx[:, :-1])
            val = rr[:, :, 1].contiguous().view(torch.float32).double()
            B = (np.float32(wl.beta).item() * m_before[w][t].double() + g[w][t].double())
            lhs = r.mom[w][t].double().pow(2).sum().item()
            rhs = B.pow(2).sum().item() - val.pow(2).sum().item()
            assert abs(lhs - rhs) <= 1e-5 * B.pow(2).sum().item()
    r.close()


def test_abi_runtime_argument_errors():
    shapes = [(64, 64)]
    tr = demo.DemoTransform(shapes, chunk=64, topk=8, beta=0.9, lr=1e-3, weight_decay=0.0, num_workers=2)
    g = [torch.zeros(64, 64, device="cuda", dtype=torch.bfloat16)]
    m = [torch.zeros(64, 64, device="cuda")]
    p = torch.zeros(tr.payload_bytes + 16, dtype=torch.uint8, device="cuda")
    with pytest.raises(demo.DemoError) as e:
        tr.compress(2, g, m, p)  # worker out of range
    assert e.value.status == 1
    with pytest.raises(demo.DemoError) as e:
        tr.compress(0, g, m, p[4:])  # misaligned payload
    assert e.value.status == 1
    with pytest.raises(demo.DemoError) as e:
        tr.decode_apply([p], m)  # n_payloads != W
    assert e.value.status == 1
    tr.compress(0, g, m, p)
    assert tr.device_status() == 0
    tr.close()


def test_binding_refuses_tensors_of_the_wrong_layout():
    shapes = [(64, 128)]
    tr = demo.DemoTransform(shapes, chunk=64, topk=8, beta=0.9, lr=1e-3, weight_decay=0.0, num_workers=1)
    g = [torch.zeros(64, 128, device="cuda", dtype=torch.bfloat16)]
    m = [torch.zeros(64, 128, device="cuda")]
    p = torch.zeros(tr.payload_bytes, dtype=torch.uint8, device="cuda")
    with pytest.raises(ValueError, match="not contiguous"):
        tr.compress(0, [torch.zeros(128, 64, device="cuda", dtype=torch.bfloat16).t()], m, p)
    with pytest.raises(ValueError, match="dtype"):
        tr.compress(0, [g[0].float()], m, p)
    with pytest.raises(ValueError, match="shape"):
        tr.compress(0, g, [torch.zeros(128, 64, device="cuda")], p)
    with pytest.raises(ValueError, match="expected cuda:0"):
        tr.compress(0, g, [torch.zeros(64, 128)], p)
    with pytest.raises(ValueError, match="payload_out"):
        tr.compress(0, g, m, p[:-8])
    with pytest.raises(ValueError, match="payloads"):
        tr.decode_apply([p.cpu()], m)
    tr.compress(0, g, m, p)
    tr.decode_apply([p], m)
    assert tr.device_status() == 0
    tr.close()


def test_bad_payload_index_is_reported_not_faulted():
    shapes = [(64, 64)]
    tr = demo.DemoTransform(shapes, chunk=64, topk=4, beta=0.9, lr=1e-3, weight_decay=0.0, num_workers=1)
    x = [torch.ones(64, 64, device="cuda")]
    rec = torch.zeros(4, 2, dtype=torch.int32, device="cuda")
    rec[:, 0] = torch.tensor([0, 1, 2, 5000], dtype=torch.int32)
    tr.decode_apply([rec.view(torch.uint8).view(-1)], x)
    assert tr.device_status() == 8  # DEMO_ERR_PAYLOAD, and the status is cleared afterwards
    assert tr.device_status() == 0
    tr.close()


def test_step_host_matches_separate_calls():
    wl = inputs.small_decoder(num_workers=2)
    r = parity.Runner(wl, max_chunks=4)
    grads = [st.next() for st in r.streams]
    host = [[g.cpu().pin_memory() for g in gw] for gw in grads]
    dev = [[torch.empty_like(g) for g in gw] for gw in grads]
    mom2 = [[torch.zeros_like(m) for m in mw] for mw in r.mom]
    params2 = [p.clone() for p in r.params]
    pay2 = [torch.zeros_like(p) for p in r.payloads]
    out = torch.zeros(wl.num_workers * r.tr.payload_bytes, dtype=torch.uint8).pin_memory()
    r.tr.step_host(host, dev, mom2, pay2, params2, out)
    torch.cuda.synchronize()
    r.step(check=False, grads=grads)
    torch.cuda.synchronize()
    assert all(torch.equal(a, b) for a, b in zip(params2, r.params))
    assert all(torch.equal(a, b) for a, b in zip(pay2, r.payloads))
    assert torch.equal(out.view(wl.num_workers, -1)[1], r.payloads[1].cpu())
    r.close()


def test_one_worker_per_rank_in_a_world_of_one():
    """The deployed form (one worker per rank, NCCL all-gather of the payloads, decode on every rank)
    through a single-rank NCCL group: same bits as compress + decode called directly with W = 1."""
    import os

    import torch.distributed as dist

    from paper_2411_19870_b200.distributed import DistributedDemo

    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(35500 + (os.getpid() % 2000))
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
            dd.step(grads, mom, params)
        torch.cuda.synchronize()
        assert dd.tr.device_status() == 0
        for _ in range(2):
            r.step(check=True, grads=[grads])
        torch.cuda.synchronize()
        assert all(torch.equal(a, b) for a, b in zip(params, r.params))
        assert all(torch.equal(a, b) for a, b in zip(mom, r.mom[0]))
        assert torch.equal(dd.slices[0], r.payloads[0])
        dd.close()
    finally:
        dist.destroy_process_group()
    r.close()


@pytest.mark.parametrize("path", [None, demo.DEMO_PATH_GENERIC])
def test_cuda_graph_replay_matches_eager_calls(path):
    """The whole step (W compress calls + decode) captured into one CUDA graph after a warm-up call (which
    uploads the pointer tables) and replayed twice gives the same bits as two eager steps."""
    wl = inputs.small_decoder(num_workers=2)
    r = parity.Runner(wl, max_chunks=4, path=path)
    grads = [st.next() for st in r.streams]

    def one_step():
        for w in range(wl.num_workers):
            r.tr.compress(w, grads[w], r.mom[w], r.payloads[w])
        r.tr.decode_apply(r.payloads, r.params)

    def reset(state=None):
        for mw in r.mom:
            for m in mw:
                m.zero_()
        if state is not None:
            for p, s in zip(r.params, state):
                p.copy_(s)

    x0 = [p.clone() for p in r.params]
    one_step()
    one_step()
    torch.cuda.synchronize()
    want_x = [p.clone() for p in r.params]
    want_m = [[m.clone() for m in mw] for mw in r.mom]
    want_p = [p.clone() for p in r.payloads]
    reset(x0)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        one_step()
    reset(x0)  # capture records the launches without running them; start both replays from the same state
    for p in r.payloads:
        p.zero_()
    graph.replay()
    graph.replay()
    torch.cuda.synchronize()
    assert r.tr.device_status() == 0
    assert all(torch.equal(a, b) for a, b in zip(want_x, r.params))
    assert all(torch.equal(a, b) for aw, bw in zip(want_m, r.mom) for a, b in zip(aw, bw))
    assert all(torch.equal(a, b) for a, b in zip(want_p, r.payloads))
    r.close()


@pytest.mark.parametrize("s,k", [(64, 32), (64, 128), (32, 32), (32, 128), (128, 32), (128, 128)])
def test_decode_fan_in_64_workers(s, k):
    """Config 5's W=64 cells on the 4096 x 4096 matrix, every chunk size: one step from zero momentum (m = g),
    every worker compressed into its own payload, decode of 64 payloads checked on sampled chunks."""
    wl = inputs.stress(chunk=s, topk=k, num_workers=64, full_set=False)
    r = parity.Runner(wl, max_chunks=64 if s < 128 else 24, seed=k + s)
    r.step()
    assert r.report["decode_chunks"] == (64 if s < 128 else 24)
    r.close()


def _free_gb():
    free, _ = torch.cuda.mem_get_info()
    return free / 1e9


def test_decoder_300m_full_size_sampled():
    """Config 3 at full size (217 tensors, P = 454 M, W = 8) in the launch configuration the benchmark
    times; 12 sampled chunks per tensor and worker (first, last, 10 random), all chunks of 1-D tensors
    up to that count, plus the whole-tensor record invariants."""
    wl = inputs.decoder_300m()
    if _free_gb() < 30:
        pytest.skip("not enough free device memory")
    r = parity.Runner(wl, max_chunks=12)
    r.step()
    r.step()
    rec = r.payloads[3].view(torch.int32).view(-1, 2)
    assert rec.shape[0] == wl.records_per_worker()
    first, n_chunks, k_eff = r.layout[len(wl.shapes) - 1]  # the embedding, the largest tensor
    idx = rec[first:first + n_chunks * k_eff, 0].view(n_chunks, k_eff)
    assert idx.min().item() >= 0 and idx.max().item() < 4096 and torch.all(idx[:, 1:] > idx[:, :-1])
    r.close()


def test_decoder_1b_full_size_sampled():
    """Config 4 at full size (146 tensors, P = 1.28 G, W = 16): the benchmark's workload and launch
    configuration, 6 sampled chunks per tensor and worker."""
    wl = inputs.decoder_1b()
    if _free_gb() < 110:
        pytest.skip("not enough free device memory")
    r = parity.Runner(wl, max_chunks=6)
    r.step()
    assert r.report["chunks"] == 16 * 146 * 6
    r.close()
    torch.cuda.empty_cache()


@pytest.mark.parametrize("s", [8, 64, 128])
@pytest.mark.parametrize("alpha", [0.2, 0.0])
def test_alpha_scaled_momentum_subtraction(s, alpha):
    """Section 2.1's subtraction coefficient: the residual removes only alpha of the transmitted part."""
    shapes = [(2 * s, 4 * s), (2 * s,)]
    wl = inputs.Workload("alpha", shapes, chunk=s, topk=max(2, s // 2), num_workers=2, grad_kind="normal", grad_std=0.01)
    for path in PATHS:
        r = parity.Runner(wl, max_chunks=10**9, path=path, alpha=alpha)
        r.step()
        r.step()
        r.close()
    with pytest.raises(demo.DemoError):
        r2 = parity.Runner(wl, max_chunks=4)
        try:
            r2.tr.set_alpha(1.5)
        finally:
            r2.close()


@pytest.mark.parametrize("s", [8, 64, 128])
@pytest.mark.parametrize("agg,phi", [(1, 0), (2, 0), (0, 1), (1, 1), (2, 1)])
def test_aggregation_and_phi_variants(s, agg, phi):
    """Mean / count-normalised aggregation (Sparse Top-k Averaging) and phi = identity, both kernel
    families; workers share gradient structure so that coordinates collide across workers."""
    shapes = [(2 * s, 2 * s), (2 * s,)]
    wl = inputs.Workload("agg", shapes, chunk=s, topk=max(2, s // 4), num_workers=5, grad_kind="normal", grad_std=0.01)
    for path in PATHS:
        r = parity.Runner(wl, max_chunks=10**9, path=path, agg=agg, phi=phi)
        base = [g for g in r.streams[0].next()]
        grads = [[(b.float() + 0.3 * o.float()).to(b.dtype) for b, o in zip(base, st.next())] for st in r.streams]
        r.step(grads=grads)
        r.step(grads=grads)
        r.close()


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("s", [8, 64, 128])
def test_identity_basis(s, path):
    """Section 4.2's baseline P = I: top-k of the momentum itself, sign of the scattered sum (at s = 64
    on the tensor-core kernels by default, on the CUDA-core dense kernels when forced)."""
    shapes = [(2 * s, 3 * s), (2 * s,)]
    wl = inputs.Workload("ident", shapes, chunk=s, topk=max(2, s // 2), num_workers=3, grad_kind="normal", grad_std=0.01)
    r = parity.Runner(wl, max_chunks=10**9, basis=np.eye(s), path=path)
    r.step()
    r.step()
    assert torch.equal(r.tr.get_basis(), torch.eye(s))
    r.close()


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("s", [8, 32, 64, 128])
def test_random_orthonormal_basis_redrawn_every_step(s, path):
    """Gaussian matrix seeded by the step number, Gram-Schmidt on the device vs the oracle's own."""
    shapes = [(2 * s, 3 * s), (4 * s,)]
    wl = inputs.Workload("randp", shapes, chunk=s, topk=max(2, s // 2), num_workers=2, grad_kind="normal", grad_std=0.01)
    r = parity.Runner(wl, max_chunks=10**9, path=path)
    for step in (1, 2, 3):
        r.set_basis(gauss=inputs.basis_gaussian(step, s).numpy())
        P = r.tr.get_basis().double().numpy()
        assert np.max(np.abs(P - r.basis)) < 2e-7
        assert np.max(np.abs(P @ P.T - np.eye(s))) < 2e-6
        r.step()
    # back to the DCT (and, where there is one, to the fast kernel family)
    r.set_basis()
    r.step()
    r.close()


@pytest.mark.parametrize("k,alpha,agg,phi", [(32, None, 0, 0), (1, 0.2, 1, 1), (200, None, 2, 0), (4096, 0.5, 2, 1)])
def test_tensor_core_kernels_under_a_random_basis(k, alpha, agg, phi):
    """s = 64 with a caller-supplied basis runs on the tcgen05 kernels: odd number of chunks (the last
    pair is half empty), several tensors, bf16 gradients, k below and above 64 up to lossless, alpha and
    the aggregation / phi variants, five workers with colliding coordinates."""
    s = 64
    shapes = [(s, 3 * s), (2 * s, 2 * s), (s,)]  # 3 + 4 = 7 chunks: an odd count
    wl = inputs.Workload("tc", shapes, chunk=s, topk=k, num_workers=5, grad_kind="normal", grad_std=0.01)
    r = parity.Runner(wl, max_chunks=10**9, gauss=inputs.basis_gaussian(11, s).numpy(), alpha=alpha, agg=agg, phi=phi)
    base = [g for g in r.streams[0].next()]
    grads = [[(b.float() + 0.3 * o.float()).to(b.dtype) for b, o in zip(base, st.next())] for st in r.streams]
    before = r.tr.launch_count
    r.step(grads=grads)
    r.step(grads=grads)
    assert r.tr.launch_count - before == 2 * (wl.num_workers + 1) * 2  # 2-D list + 1-D list per call
    assert r.tr.device_status() == 0
    r.close()


@pytest.mark.parametrize("seed", range(12))
def test_randomized_tensor_core_cases(seed):
    """Seeded random configurations at s = 64 under a random orthonormal basis (tensor-core kernels), the
    basis redrawn before each of the two steps."""
    rng = np.random.default_rng(5000 + seed)
    s = 64
    k = int(rng.choice([1, 5, 31, 32, 33, 64, 65, 130, 1000, 4096]))
    W = int(rng.integers(1, 5))
    shapes = [(s * int(rng.integers(1, 4)), s * int(rng.integers(1, 4))) for _ in range(int(rng.integers(1, 4)))]
    shapes += [(s * int(rng.integers(1, 4)),) for _ in range(int(rng.integers(0, 2)))]
    dtype = torch.bfloat16 if rng.random() < 0.5 else torch.float32
    alpha = None if rng.random() < 0.5 else float(rng.choice([0.2, 0.5]))
    agg, phi = int(rng.integers(0, 3)), int(rng.integers(0, 2))
    wl = inputs.Workload("tc-random%d" % seed, shapes, chunk=s, topk=k, num_workers=W, grad_kind="tensor_scaled",
                         grad_std=0.01, grad_dtype=dtype)
    r = parity.Runner(wl, max_chunks=10**9, seed=seed, alpha=alpha, agg=agg, phi=phi)
    for step in (1, 2):
        r.set_basis(gauss=inputs.basis_gaussian(100 * seed + step, s).numpy())
        r.step()
    r.close()


@pytest.mark.parametrize("basis_kind", ["identity", "random"])
def test_tensor_core_kernels_on_tie_maker_chunks(basis_kind):
    """All-zero, constant, symmetric and +-a tiles (the stress configuration's tie-makers, here in 30 % of the
    chunks) through the tensor-core kernels: under the identity basis the ties survive the transform, so the
    candidate path overflows and the radix select with the index tie-break has to take over."""
    s = 64
    wl = inputs.Workload("tc-ties", [(4 * s, 4 * s), (2 * s, 3 * s)], chunk=s, topk=32, num_workers=3,
                         grad_kind="student_t_ties", grad_std=1e-3)
    kw = dict(basis=np.eye(s)) if basis_kind == "identity" else dict(gauss=inputs.basis_gaussian(3, s).numpy())
    r = parity.Runner(wl, max_chunks=10**9, **kw)
    for st in r.streams:
        st.tie_fraction = 0.3
    r.step()
    r.step()
    r.close()


def test_basis_argument_errors_keep_the_previous_basis():
    s = 8
    wl = inputs.Workload("basis-err", [(2 * s, 2 * s)], chunk=s, topk=4, num_workers=1, grad_kind="normal", grad_std=0.01)
    r = parity.Runner(wl, max_chunks=10**9, gauss=inputs.basis_gaussian(7, s).numpy())
    before = r.tr.get_basis()
    with pytest.raises(demo.DemoError):
        r.tr.set_basis(torch.ones((s, s)))  # rows not orthonormal
    with pytest.raises(demo.DemoError):
        r.tr.set_basis_gaussian(torch.ones((s, s)))  # singular: the second row has nothing left
    with pytest.raises(ValueError):
        r.tr.set_basis(torch.eye(s + 1))
    assert torch.equal(r.tr.get_basis(), before)
    r.step()
    r.close()


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("s", [8, 32, 64, 128])
def test_nan_and_inf_gradients_neither_hang_nor_corrupt_other_tensors(s, path):
    """Results for chunks that contain NaN or Inf are unspecified, but the kernels must finish, every
    chunk must still carry k_eff records with distinct, ascending, in-range indices (a consumer relies on
    that), and tensors without such values must come out bit-identical to a clean run."""
    shapes = [(2 * s, 2 * s), (2 * s, 4 * s), (2 * s,), (4 * s,)]
    wl = inputs.Workload("nonfinite", shapes, chunk=s, topk=8, num_workers=2, grad_kind="normal", grad_std=0.01)
    clean = parity.Runner(wl, max_chunks=10**9, path=path)
    dirty = parity.Runner(wl, max_chunks=10**9, path=path)
    grads = [st.next() for st in clean.streams]
    bad = [[g.clone() for g in gw] for gw in grads]
    for w in range(wl.num_workers):
        bad[w][0][3, 5] = float("nan")          # one chunk of the first matrix
        bad[w][0][s + 1, s + 2] = float("inf")  # another one
        bad[w][0][s + 7, 9] = float("-inf")     # and a third
        bad[w][2][3] = float("nan")             # one segment of the first vector
    clean.step(check=True, grads=grads)
    dirty.step(check=False, grads=bad)
    torch.cuda.synchronize()
    assert dirty.tr.device_status() == 0
    for tns in (1, 3):  # untouched tensors: same bits as the clean run
        assert torch.equal(clean.params[tns], dirty.params[tns])
        for w in range(wl.num_workers):
            assert torch.equal(clean.mom[w][tns], dirty.mom[w][tns])
    for w in range(wl.num_workers):
        raw = dirty.payloads[w].cpu().numpy().view(parity.orc.RECORD_DTYPE)
        for tns, shp in enumerate(shapes):
            first, n_chunks, k_eff = dirty.layout[tns]
            idx = raw["idx"][first:first + n_chunks * k_eff].reshape(n_chunks, k_eff)
            M = s * s if len(shp) == 2 else s
            assert idx.min() >= 0 and idx.max() < M
            assert np.all(np.diff(idx, axis=1) > 0)
    clean.close()
    dirty.close()


def test_bounded_wait_expires_into_a_status_and_the_context_survives():
    """Failure detection without a GPU fault: a wait that nothing satisfies runs out after ~1 ms, the
    kernel returns, the sticky status says TIMEOUT, and the same context then computes correctly."""
    wl = inputs.small_decoder(num_workers=2)
    r = parity.Runner(wl, max_chunks=16)
    r.step()
    r.tr.selftest_bounded_wait(2_000_000)  # ~1 ms of SM clock
    assert r.tr.device_status() == 7       # DEMO_ERR_TIMEOUT ...
    assert r.tr.device_status() == 0       # ... reported once, then cleared
    r.step()                               # parity-checked step on the same context
    r.close()


@pytest.mark.parametrize("s,basis", [(32, None), (64, None), (128, None), (64, "random")])
def test_untouched_tiles_among_ordinary_ones(s, basis):
    """Row blocks whose gradient is exactly zero on a zero momentum (embedding rows of tokens that did not occur):
    their chunks take the all-zero shortcut of the fast, s = 128 and tensor-core kernels while their neighbours
    go through the ordinary selection; every chunk is checked against the oracle, two steps."""
    wl = inputs.Workload("zero-rows", [(6 * s, 4 * s), (3 * s, 5 * s)], chunk=s, topk=min(32, s), num_workers=2,
                         grad_kind="normal", grad_std=1e-3)
    kw = dict(gauss=inputs.basis_gaussian(9, s).numpy()) if basis else {}
    r = parity.Runner(wl, max_chunks=10**9, **kw)
    for step in range(2):
        grads = [st.next() for st in r.streams]
        for g in grads:
            g[0][s:3 * s] = 0          # two chunk rows of the first tensor
            g[1][:, 2 * s:3 * s] = 0   # one chunk column of the second
        r.step(grads=grads)
    # the zero chunks' records are the lowest indices with value 0
    first, n_chunks, k_eff = r.layout[0]
    rec = parity.gather_records(r.payloads[0], first, k_eff, np.arange(4, 12, dtype=np.int64))
    assert np.array_equal(rec["idx"], np.tile(np.arange(k_eff, dtype=np.int32), (8, 1))) and np.all(rec["val"] == 0)
    r.close()


@pytest.mark.parametrize("s", [32, 64, 128])
@pytest.mark.parametrize("pattern", ["rows", "cols"])
def test_tiles_of_low_rank(s, pattern):
    """Gradient tiles with one to three active rows (embedding gradients: only the tokens of the batch have a
    row) or columns (output layer): the row maxima bound the k-th coefficient loosely there, the candidate
    lists run long, and the kernels' wide-list / radix paths decide.  Every chunk against the oracle."""
    shape = (6 * s, 5 * s)
    wl = inputs.Workload("low-rank", [shape], chunk=s, topk=min(32, s), num_workers=2, grad_kind="normal", grad_std=1e-3)
    r = parity.Runner(wl, max_chunks=10**9)
    gen = torch.Generator(device="cuda")
    gen.manual_seed(5)
    for step in range(2):
        grads = []
        for w in range(2):
            g = torch.zeros(shape, device="cuda")
            for b in range(shape[0] // s if pattern == "rows" else shape[1] // s):
                n_act = 1 + (b + w + step) % 3
                idx = torch.randperm(s, generator=gen, device="cuda")[:n_act] + b * s
                if pattern == "rows":
                    g[idx] = torch.randn((n_act, shape[1]), generator=gen, device="cuda") * 1e-3
                else:
                    g[:, idx] = torch.randn((shape[0], n_act), generator=gen, device="cuda") * 1e-3
            grads.append([g.to(torch.bfloat16)])
        r.step(grads=grads)
    r.close()
