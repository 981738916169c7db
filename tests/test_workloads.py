"""The seeded input generators: shapes, determinism, grids, distinct pools."""
import numpy as np
import pytest

from paper_2604_11109_b200 import workloads as w


@pytest.mark.parametrize("cfg", [1, 2, 3, 4, 5])
def test_shapes_dtypes_and_determinism(cfg):
    c = w.get_config(cfg, m=512, batch=2 if cfg == 3 else None, n=128 if cfg == 5 else None)
    a, b = w.generate(c), w.generate(c)
    assert a["X"].shape == (c.batch, c.n, c.d) and a["Xcand"].shape == (c.batch, c.m, c.d)
    assert a["y"].shape == (c.batch, c.n) and a["ell"].shape == (c.batch, c.d)
    for k in a:
        assert a[k].dtype == np.float32
        assert np.array_equal(a[k], b[k])
    assert np.all(np.isfinite(a["X"])) and np.all(np.isfinite(a["y"]))
    assert np.all(a["ell"] >= c.ell_lo) and np.all(a["ell"] <= c.ell_hi)
    assert abs(float(a["y"][0].mean())) < 1e-5 and abs(float(a["y"][0].std()) - 1) < 1e-4
    assert a["sn2"][0] == np.float32(c.noise_var) and a["sf2"][0] == 1
    # pool rows are distinct
    assert np.unique(a["Xcand"][0], axis=0).shape[0] == c.m
    assert np.unique(a["X"][0], axis=0).shape[0] == c.n


def test_grid_features_take_only_grid_values():
    c = w.get_config(2, m=2048)
    g = w.generate(c)
    for j, lv in enumerate(w.feature_levels(c)):
        assert set(np.unique(g["Xcand"][0][:, j])).issubset(set(lv.astype(np.float32)))


def test_permutation_rows_are_unit_norm_one_hot():
    c = w.get_config(4, m=256, n=64)
    g = w.generate(c)
    xc = g["Xcand"][0].reshape(c.m, 32, 4)
    assert np.all((xc > 0).sum(axis=2) == 1)
    assert np.allclose((g["Xcand"][0] ** 2).sum(axis=1), 1.0, atol=1e-6)
    # each position bucket holds exactly 8 passes
    assert np.all((xc > 0).sum(axis=1) == 8)


def test_batched_gps_differ_and_stress_twin_has_near_neighbours():
    c = w.get_config(3, m=64, batch=3)
    g = w.generate(c)
    assert not np.array_equal(g["X"][0], g["X"][1]) and not np.array_equal(g["ell"][0], g["ell"][2])
    cs = w.get_config(1, stress=True)
    gs = w.generate(cs)
    d2 = ((gs["Xcand"][0][:, None, :] - gs["X"][0][None, :, :]) ** 2).sum(-1).min(axis=1)
    assert (d2 < 0.05).sum() >= cs.m // 16
    assert np.all(gs["ell"] >= cs.ell_lo)


def test_sample_indices_sorted_distinct():
    c = w.get_config(5)
    s = w.sample_indices(c, 8192)
    assert s.shape == (8192,) and np.all(np.diff(s) > 0) and s[-1] < c.m


def test_tpe_levels_mark_binary_flags_and_grids():
    from paper_2604_11109_b200 import workloads as w
    c2, c5, c4 = w.get_config(2), w.get_config(5), w.get_config(4)
    lv2 = w.tpe_levels(c2)
    assert lv2.tolist() == [0, 0, 0, 0, 0, 2] + [2] * 10           # five launch parameters, one bool, ten flags
    assert w.tpe_levels(c5).tolist() == [0] * 32 + [2] * 32
    assert w.tpe_levels(c4).tolist() == [0] * 128
    g2 = w.tpe_levels(c2, grid=True)
    assert g2[:6].tolist() == [-32, -8, -4, 0, 0, 2]               # equally spaced levels become grids; 224 levels
    assert w.tpe_levels(c5, grid=True).tolist() == [-16] * 32 + [2] * 32   # and unevenly spaced ones stay ordinal
    # the declared grids are the generator's own values
    for l, code in zip(w.feature_levels(c2), g2):
        if code < 0:
            assert np.array_equal(np.float32(l), np.float32(np.arange(-code) / (-code - 1)))
