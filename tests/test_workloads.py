"""The synthetic workloads: segment tables and value structure (CPU only)."""
import pytest
import torch

import workloads as wlmod


def test_resnet_segment_tables():
    r18, r50 = wlmod.resnet18_sizes(), wlmod.resnet50_sizes()
    assert (len(r18), sum(r18)) == (62, 11_689_512)
    assert (len(r50), sum(r50)) == (161, 25_557_032)
    assert sum(s.k for s in wlmod.segment_table(r18, 1, 100)) == 116_928
    assert sum(s.k for s in wlmod.segment_table(r50, 1, 1000)) == 25_670
    assert wlmod.kept_count(1_048_576, 1, 100) == 10_486
    assert sum(wlmod.lstm_lm_sizes()) == 66_034_000


def test_resnet_sizes_agree_with_torchvision():
    tv = pytest.importorskip("torchvision")
    assert wlmod.resnet18_sizes() == [p.numel() for p in tv.models.resnet18(weights=None).parameters()]
    assert wlmod.resnet50_sizes() == [p.numel() for p in tv.models.resnet50(weights=None).parameters()]


def test_generators_are_seeded_and_shaped():
    wl = wlmod.workload("c1")
    a = wlmod.generate(wl, 0, 0, "cpu", sizes=[4096])
    b = wlmod.generate(wl, 0, 0, "cpu", sizes=[4096])
    c = wlmod.generate(wl, 1, 0, "cpu", sizes=[4096])
    assert torch.equal(a, b) and not torch.equal(a, c)
    assert abs(a.std().item() - 1e-3) < 1e-4

    sizes = [650 * 40, 1000, 1000, 650 * 40, 40, 500]
    g = wlmod.generate(wlmod.workload("c4"), 0, 0, "cpu", sizes=sizes)
    rows = g[:650 * 40].view(40, 650)
    zero_rows = (rows == 0).all(dim=1)
    assert zero_rows.sum() >= 30
    assert ((rows != 0).all(dim=1) | zero_rows).all()
    assert not (g.view(torch.int32) == -2 ** 31).any()      # no negative zeros

    t = wlmod.generate(wlmod.workload("c5"), 0, 0, "cpu", sizes=[200_000])
    assert t.abs().max() > 20e-3                             # heavy tail
    assert torch.isfinite(t).all()

    ints = wlmod.gen_small_integers(1000, wlmod.make_generator(0, 0, 0, "cpu"), "cpu")
    assert torch.equal(ints, ints.round()) and ints.abs().max() <= 1024


def test_segment_scales_span_orders_of_magnitude():
    sizes = [512] * 30
    g = wlmod.generate(wlmod.workload("c3"), 0, 0, "cpu", sizes=sizes).view(30, 512)
    s = g.abs().mean(dim=1)
    assert s.max() / s.min() > 30
