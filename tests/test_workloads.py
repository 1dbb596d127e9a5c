"""The seeded input generators: shapes, ranges and determinism of the five
benchmark configurations (no solver arithmetic is involved)."""
import numpy as np
import pytest

from paper_2407_14843_b200 import workloads as W

EXPECT = {  # cfg: (N, S, C, |B|, H, T, K, cells per instance)
    1: (64, 3, 8, 4, 4, 500, 128, 251_502),
    2: (4096, 5, 16, 6, 16, 1000, 1536, 2_006_004),
    3: (86400, 10, 32, 6, 8, 800, 192, 2_890_809),
    4: (16384, 8, 64, 7, 32, 4000, 14336, 56_042_007),
    5: (4096, 20, 64, 8, 64, 8192, 32768, 637_767_699),
}


@pytest.mark.parametrize("cfg", sorted(EXPECT))
def test_config_shapes(cfg):
    n = None if cfg in (1, 2, 3) else 256
    wl = W.make_workload(cfg, n)
    N, S, C, nb, H, T, K, cells = EXPECT[cfg]
    assert wl.n_instances == (N if n is None else n)
    assert (wl.n_stages, wl.c_max, wl.n_batch, wl.h_max, wl.T) == (S, C, nb, H, T)
    assert wl.n_candidates == K and wl.minplus_cells == cells
    assert wl.lat_us.shape == (wl.n_profiles, S, C, nb) and wl.lat_us.dtype == np.int32
    assert (wl.lat_us >= 1000).all() and (wl.lat_us % 1000 == 0).all()
    # latency falls with cores and grows with batch size
    assert (np.diff(wl.lat_us, axis=2) <= 0).all() and (np.diff(wl.lat_us, axis=3) >= 0).all()
    assert wl.lambda_mrps.dtype == np.uint32 and (wl.lambda_mrps >= 1000).all()
    assert (wl.profile_id >= 0).all() and (wl.profile_id < wl.n_profiles).all()
    assert wl.vertical == (cfg == 3)
    if wl.vertical:
        assert wl.replicas.shape == (wl.n_instances, S)
        assert (wl.replicas >= 1).all() and (wl.replicas <= H).all()
        assert (wl.replicas == wl.replicas[0]).all()


def test_generators_are_counter_based():
    a = W.make_workload(4, 64)
    b = W.make_workload(4, 256)
    assert np.array_equal(a.lambda_mrps, b.lambda_mrps[:64])
    assert np.array_equal(a.lat_us, b.lat_us)
    c = W.make_workload(4, 64, seed_offset=1)
    assert not np.array_equal(a.lambda_mrps, c.lambda_mrps)
    assert a.checksums() == W.make_workload(4, 64).checksums()
    assert a.checksums() != c.checksums()


def test_rate_processes():
    r2 = W.make_workload(2).lambda_mrps / 1000.0
    assert 60 < np.median(r2) < 170 and r2.min() >= 1 and r2.max() <= 2000
    z = np.log(r2)
    assert np.corrcoef(z[:-1], z[1:])[0, 1] > 0.7           # bursty: neighbours correlate
    r3 = W.make_workload(3).lambda_mrps / 1000.0
    assert 19.9 < r3.min() < 25 and r3.max() > 400          # diurnal base plus spikes
    assert abs(r3[43200] / 400.0 - 1) < 0.01 or r3[43200] > 1000
    r4 = W.make_workload(4, 4096).lambda_mrps / 1000.0
    assert 250 < np.median(r4) < 360
    r5 = W.make_workload(5, 4096).lambda_mrps / 1000.0
    assert 800 < np.median(r5) < 1250 and r5.max() <= 20000


def test_uniform_and_normal_draws():
    i = np.arange(200000, dtype=np.uint64)
    u = W.rand_uniform(1, 2, i)
    assert 0 <= u.min() and u.max() < 1 and abs(u.mean() - 0.5) < 0.005
    z = W.rand_normal(1, 3, i)
    assert abs(z.mean()) < 0.01 and abs(z.std() - 1) < 0.01
    k = W.rand_int(1, 4, i, 3, 7)
    assert set(np.unique(k)) == {3, 4, 5, 6, 7}
