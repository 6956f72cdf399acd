"""Pins for the oracle's seeded k-means++ start (a draw proportional to the squared distance to the
nearest start point so far, written as an exponential race over counter-based uniforms)."""
import numpy as np

from oracle import muse_oracle as orc


def test_uniforms_are_seeded_distinct_and_inside_the_unit_interval():
    u = orc._kpp_uniforms(4096, 3, 17, 2)
    assert u.min() > 0 and u.max() < 1
    assert abs(u.mean() - 0.5) < 0.02 and abs(u.var() - 1 / 12) < 0.005
    np.testing.assert_array_equal(u, orc._kpp_uniforms(4096, 3, 17, 2))
    for other in (orc._kpp_uniforms(4096, 4, 17, 2), orc._kpp_uniforms(4096, 3, 18, 2), orc._kpp_uniforms(4096, 3, 17, 3)):
        assert (other != u).mean() > 0.99
    # every value is k + 1/2 over 2^23: exact in single precision too
    assert np.array_equal(u.astype(np.float32).astype(np.float64), u)
    assert np.array_equal(u * 2 ** 23 - 0.5, np.round(u * 2 ** 23 - 0.5))


def test_draw_frequencies_follow_the_squared_distances():
    """The race must pick index t with probability d2_t / sum(d2): chi-square against that law over
    many seeds (a wrong race, e.g. the largest d2 * e or d2 / u, fails by a wide margin)."""
    d2 = np.array([0.0, 1.0, 4.0, 0.5, 2.5, 0.0, 8.0])
    trials = 6000
    hits = np.zeros(7)
    for s in range(trials):
        hits[orc.kmeanspp_step(d2, 1 + s % 5, 1000 + s, s % 3)[0]] += 1
    expect = trials * d2 / d2.sum()
    assert hits[0] == 0 and hits[5] == 0
    nz = d2 > 0
    chi2 = ((hits[nz] - expect[nz]) ** 2 / expect[nz]).sum()
    assert chi2 < 20.5                                      # 4 degrees of freedom, p = 4e-4


def test_start_indices_are_distinct_seeded_and_begin_at_the_shuffle():
    rng = np.random.default_rng(5)
    X = rng.standard_normal((300, 4))
    i1 = orc.kmeanspp_init(X, 40, 9, 1)
    assert len(set(i1.tolist())) == 40 and i1.dtype == np.int32
    assert i1[0] == orc.feistel_permute(0, 300, 9, 1)
    np.testing.assert_array_equal(i1, orc.kmeanspp_init(X, 40, 9, 1))
    assert (orc.kmeanspp_init(X, 40, 10, 1) != i1).any() and (orc.kmeanspp_init(X, 40, 9, 2) != i1).any()
    # the potential (sum of squared distances to the nearest start) never grows, and each drawn point had d2 > 0
    d2 = ((X - X[i1[0]]) ** 2).sum(1)
    for c in range(1, 40):
        assert d2[i1[c]] > 0
        nd = np.minimum(d2, ((X - X[i1[c]]) ** 2).sum(1))
        assert nd.sum() <= d2.sum()
        d2 = nd


def test_one_start_per_separated_blob():
    rng = np.random.default_rng(6)
    centres = 100.0 * np.eye(6)
    lab = rng.integers(0, 6, 240)
    X = centres[lab] + 0.01 * rng.standard_normal((240, 6))
    for seed in range(5):
        idx = orc.kmeanspp_init(X, 6, seed, 0)
        assert sorted(lab[idx].tolist()) == list(range(6))


def test_all_points_equal_falls_back_to_the_lowest_index():
    idx, keys = orc.kmeanspp_step(np.zeros(5), 1, 0, 0)
    assert idx == 0 and (keys == 0).all()
