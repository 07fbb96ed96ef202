"""The seeded workload generators: shapes and sizes of the five configurations, determinism."""
import torch

from paper_2411_19870_b200 import inputs


def test_workload_sizes():
    t = inputs.tiny()
    assert t.n_params == 131_584 and t.records_per_worker() == 8448
    s = inputs.single_matrix()
    assert s.n_params == 67_108_864 and s.n_chunks() == 16_384 and s.records_per_worker() == 524_288
    a = inputs.decoder_300m()
    assert len(a.shapes) == 217 and a.n_params == 454_213_632 and a.records_per_worker() == 3_572_736
    b = inputs.decoder_1b()
    assert len(b.shapes) == 146 and b.n_params == 1_279_852_544 and b.records_per_worker() == 10_031_104
    assert b.n_chunks() == 312_448 + 1024


def test_streams_are_seeded_and_worker_specific():
    wl = inputs.tiny()
    a = inputs.GradStream(wl, 0, "cpu").next()
    b = inputs.GradStream(wl, 0, "cpu").next()
    c = inputs.GradStream(wl, 1, "cpu").next()
    assert all(torch.equal(x, y) for x, y in zip(a, b))
    assert not torch.equal(a[0], c[0])
    assert a[0].dtype == torch.float32 and a[0].shape == (256, 512)
    assert abs(a[0].std().item() - 0.01) < 1e-3


def test_tie_maker_chunks_exist():
    wl = inputs.stress(chunk=32, topk=8, num_workers=1, full_set=False)
    g = inputs.GradStream(wl, 0, "cpu").next()[0].float().view(128, 32, 128, 32).permute(0, 2, 1, 3)
    zero = (g.abs().amax(dim=(2, 3)) == 0).sum().item()
    const = ((g.amax(dim=(2, 3)) == g.amin(dim=(2, 3))) & (g.abs().amax(dim=(2, 3)) > 0)).sum().item()
    assert zero > 50 and const > 50
