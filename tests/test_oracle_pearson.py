"""Pins of the oracle's maximum Pearson correlation (Appendix A, Eq. 4) against what the mathematics fixes."""
import numpy as np

import oracle
from paper_2501_14183_b200 import inputs


def test_matches_numpy_corrcoef():
    rng = np.random.default_rng(3)
    x = rng.normal(size=(3, 17, 96)).astype(np.float32)
    x[:, 5] = 0.7 * x[:, 2] + 0.1 * rng.normal(size=(3, 96))          # one strongly correlated pair
    got = oracle.pearson_max(x)
    for b in range(3):
        c = np.corrcoef(x[b].astype(np.float64))
        np.fill_diagonal(c, -np.inf)
        np.testing.assert_allclose(got[b], c.max(axis=1), rtol=0, atol=1e-12)


def test_closed_forms():
    t = np.arange(96)
    base = np.sin(2 * np.pi * 4 * t / 96)
    x = np.stack([base,                       # 0
                  3.0 * base + 5.0,           # 1: positive affine image of 0 -> rho = 1
                  -2.0 * base + 1.0,          # 2: negative affine image -> rho = -1 with 0 and 1
                  np.sin(2 * np.pi * 7 * t / 96),     # 3: another integer bin -> orthogonal to 0, 1, 2 (rho = 0)
                  np.cos(2 * np.pi * 4 * t / 96),     # 4: same bin in quadrature -> rho = 0 with 0, 1, 2 as well
                  np.full(96, 2.5)])[None].astype(np.float32)   # 5: constant -> rho = 0 with everything
    got = oracle.pearson_max(x)[0]
    np.testing.assert_allclose(got[[0, 1]], 1.0, atol=1e-6)
    np.testing.assert_allclose(got[2], 0.0, atol=1e-6)          # its best partner is an orthogonal one, not the anti-correlated pair
    np.testing.assert_allclose(got[[3, 4, 5]], 0.0, atol=1e-6)


def test_mixture_has_the_textbook_coefficient():
    # w = a u + b e with u, e orthogonal and of equal norm  ->  rho(u, w) = a / sqrt(a^2 + b^2)
    t = np.arange(96)
    u, e = np.sin(2 * np.pi * 3 * t / 96), np.sin(2 * np.pi * 11 * t / 96)
    a, b = 0.8, 0.6
    x = np.stack([u, a * u + b * e])[None].astype(np.float32)
    got = oracle.pearson_max(x)[0]
    np.testing.assert_allclose(got, a / np.hypot(a, b), atol=1e-6)


def test_invariances_and_single_variate():
    rng = np.random.default_rng(5)
    x = rng.normal(size=(2, 9, 48)).astype(np.float32)
    ref = oracle.pearson_max(x)
    scaled = (x.astype(np.float64) * rng.uniform(0.5, 3.0, size=(2, 9, 1)) + rng.normal(size=(2, 9, 1))).astype(np.float32)
    np.testing.assert_allclose(oracle.pearson_max(scaled), ref, atol=2e-6)       # positive scale and shift per variate
    perm = rng.permutation(9)
    np.testing.assert_allclose(oracle.pearson_max(x[:, perm]), ref[:, perm], atol=1e-12)   # variates relabelled
    assert np.all(oracle.pearson_max(x[:, :1]) == -2.0)                          # no other variate


def test_synthetic_workloads_are_redundant_like_the_paper_says():
    # Sec. 1: 79.4 % (Electricity) and 94.7 % (Traffic) of the variates have a partner above 0.9; the synthetic stand-ins
    # are built to be redundant in the same way (a loose check of the generator, instance by instance)
    for name, floor in (("elec", 0.6), ("traffic", 0.8)):
        w = inputs.WORKLOADS[name]
        x = inputs.make_windows(w, B=2)
        share = (oracle.pearson_max(x) > 0.9).mean()
        assert share >= floor, (name, share)
