"""The seeded generators are reproducible and have the shapes and densities the configs name."""
import numpy as np

from paper_2609_25869_b200 import inputs as I


def test_generators_are_deterministic_and_shaped():
    a, b = I.config_tiny(), I.config_tiny()
    assert np.array_equal(a.mask, b.mask) and a.mask.shape == (2, 32, 32)
    assert (a.mask[:, np.arange(32), np.arange(32)] == 1).all()
    assert 0.2 < a.mask.mean() < 0.35
    m = I.config_mid()
    assert m.mask.shape == (8, 128, 128) and abs(m.mask.sum(axis=2).mean() - 19.4) < 0.5
    q1, _, _ = a.qkv()
    q2, _, _ = b.qkv()
    assert q1.dtype.is_floating_point and bool((q1 == q2).all())
    assert abs(float(q1.float().std()) - 1.0) < 0.02


def test_stress_masks():
    s = I.config_stress_a(H=1, N=4096)
    assert s.mask.shape == (1, 256, 64)
    assert (s.mask.sum(axis=2) == round(0.15 * 64)).all()          # density target per row
    b = I.config_stress_b(H=2, N=4096)
    assert b.mask.shape == (2, 16, 16) and (b.mask[:, np.arange(16), np.arange(16)] == 1).all()


def test_sweep_request_hits_its_density_and_skew():
    r = I.config_sweep(7, H=8, B=(128, 128), rho=0.10)
    assert r.mask.shape == (8, 591, 591)
    assert abs(r.mask.mean() - 0.10) < 0.02
    per_head = r.mask.mean(axis=(1, 2))
    assert per_head.max() / per_head.min() > 5      # one heavy head
    assert (r.mask.sum(axis=2) >= 1).all()
    # the block of each row's own tile is always active (window priority, nearest first)
    assert (r.mask[:, np.arange(591), np.arange(591)] == 1).all()


def test_sample_query_blocks():
    s = I.sample_query_blocks(1, 3, 900, 64)
    assert all(len(set(v.tolist())) == 64 and v.max() < 900 for v in s.values())
    assert not np.array_equal(s[0], s[1])
    assert np.array_equal(I.sample_query_blocks(1, 2, 10, 64)[0], np.arange(10))
