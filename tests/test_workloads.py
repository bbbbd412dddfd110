"""The seeded input generators: shapes, determinism and the stated structure."""
import numpy as np
import torch

from paper_2011_06495_b200 import workloads as WL


def test_named_configs_have_the_stated_sizes():
    c2, c3, c4 = (WL.resnet_like(n) for n in ("c2", "c3", "c4"))
    assert (c2.N, c2.d, c2.K, c2.steps) == (10, 11_173_962, 111_739, 20)
    assert (c3.N, c3.d, c3.K, c3.steps) == (25, 11_173_962, 11_173, 20)
    assert (c4.N, c4.d, c4.K, c4.steps) == (8, 25_557_032, 6_389, 50)
    cells = WL.sweep_cells()
    assert len(cells) == 27
    assert {(w.N, w.d) for w in cells} == {(N, d) for N in (4, 16, 64) for d in (1 << 20, 1 << 24, 1 << 27)}
    assert sorted({w.K for w in cells if w.d == 1 << 20}) == [262, 1048, 10485]


def test_segments_partition_the_row():
    for name in ("c2", "c4"):
        w = WL.resnet_like(name)
        bounds, std = WL.layer_segments(w)
        assert bounds[0] == 0 and bounds[-1] == w.d and len(std) == w.segments
        assert np.all(np.diff(bounds) >= 16)
        assert std.min() >= w.std_lo * 0.999 and std.max() <= w.std_hi * 1.001
        b2, s2 = WL.layer_segments(w)
        assert np.array_equal(bounds, b2) and np.array_equal(std, s2)


def test_gradients_are_deterministic_and_structured():
    w = WL.scaled(WL.resnet_like("c3"), d=40_000, N=6)
    a = WL.gradients(w, 3)
    b = WL.gradients(w, 3)
    c = WL.gradients(w, 4)
    assert a.shape == (6, 40_000) and a.dtype == torch.float32
    assert torch.equal(a, b) and not torch.equal(a, c)
    # half of the variance is shared: rows correlate at about 0.5 once rescaled by the layer std
    z = a / WL.std_vector(w)
    r = np.corrcoef(z.numpy())
    off = r[~np.eye(6, dtype=bool)]
    assert 0.4 < off.mean() < 0.6


def test_c1_variants():
    free = WL.gradients(WL.resnet_like("c1"), 0)
    assert all(torch.unique(free[n].abs()).numel() == free.shape[1] for n in range(free.shape[0]))
    tied = WL.gradients(WL.resnet_like("c1_ties"), 0)
    assert torch.equal(tied, (tied * 10).round() / 10)
    assert torch.unique(tied.abs()).numel() < 100


def test_student_t_is_heavy_tailed():
    w = WL.scaled(WL.resnet_like("c4"), d=200_000, N=2)
    g = WL.gradients(w, 0) / WL.std_vector(w)
    kurt = float(((g - g.mean()) ** 4).mean() / g.var() ** 2)
    assert kurt > 6.0                       # a Gaussian has 3


def test_sweep_error_buffer_is_seeded_noise():
    w = WL.scaled(WL.sweep_cells()[0], d=50_000)
    e = WL.initial_err(w)
    assert abs(float(e.std()) - 0.01) < 1e-3 and torch.equal(e, WL.initial_err(w))
