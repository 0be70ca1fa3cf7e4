"""Pins for the skew model: Algorithm 1 against the closed-form inverse of the
symmetric Dirichlet's expected sum of squares, ddist:X end points, and exemplar
properties (Sections III-A, IV-A)."""
import numpy as np
import pytest

import damoe_inputs as di
from oracle import modeling


def test_eff_exp_of_probability_vectors():
    assert modeling.eff_exp(np.full(256, 1 / 256)) == pytest.approx(256.0, rel=1e-12)
    e1 = np.zeros(256)
    e1[3] = 1.0
    assert modeling.eff_exp(e1) == 1.0
    p = np.array([0.5, 0.25, 0.25])
    assert modeling.eff_exp(p) == pytest.approx(1 / (0.25 + 0.0625 + 0.0625))


def test_ddist_end_points():
    assert modeling.ddist_target(256, 1) == 256
    assert modeling.ddist_target(256, 256) == 1
    assert modeling.ddist_target(384, 1.5) == 256


def test_eff_exp_increases_with_alpha():
    draw = di.dirichlet_sampler(0)
    vals = [np.mean([modeling.eff_exp(p) for p in draw(a, 256, 64)]) for a in (0.05, 0.2, 1.0, 10.0)]
    assert all(b > a for a, b in zip(vals, vals[1:]))
    # E[1/sum p^2] >= 1/E[sum p^2] = (E a + 1)/(a + 1): 13.1, 43.5, 128.5, 232.8
    for v, a in zip(vals, (0.05, 0.2, 1.0, 10.0)):
        closed = (256 * a + 1) / (a + 1)
        assert closed * 0.97 < v < closed * 1.25


@pytest.mark.parametrize("X,alpha_closed", [(1.1, 9.96), (1.5, 1.99), (2.0, 0.99), (4.0, 0.33)])
def test_algorithm1_matches_closed_form_inverse(X, alpha_closed):
    E = 256
    target = modeling.ddist_target(E, X)
    a = modeling.binary_search_alpha(target, E, S=64, iters=60, draw=di.dirichlet_sampler(0))
    # closed form: alpha ~ (eff - 1) / (E - eff); sampling noise and Jensen gap allowed for
    assert a == pytest.approx((target - 1) / (E - target), rel=0.12)
    assert a == pytest.approx(alpha_closed, rel=0.15)
    # round trip: the found alpha reproduces the target (rejection sampling makes v(alpha) only piecewise smooth)
    v = np.mean([modeling.eff_exp(p) for p in di.dirichlet_sampler(0)(a, E, 64)])
    assert v == pytest.approx(target, rel=2e-2)


def test_algorithm1_is_monotone_in_target_and_saturates():
    draw = di.dirichlet_sampler(1)
    a = [modeling.binary_search_alpha(t, 64, 32, 50, draw) for t in (4, 16, 48)]
    assert a[0] < a[1] < a[2]
    # X = 1 (target = E) is unreachable for finite alpha: search runs to the top of its range
    assert modeling.binary_search_alpha(64, 64, 16, 40, draw) > 1e5


def test_algorithm1_steps_by_hand():
    # a fake sampler whose eff_exp equals alpha exactly: bisection on [1e-6, 1e6]
    def draw(alpha, E, S):
        p = np.zeros((S, E))
        m = max(1, min(E, int(round(alpha))))
        p[:, :m] = 1.0 / m
        return p
    # target 32.5 separates m = 32 from m = 33, i.e. alpha = 32.5; 30 halvings of
    # [1e-6, 1e6] leave an interval of 1e6 / 2^30 < 1e-3 around it
    a = modeling.binary_search_alpha(32.5, 1000, 3, 30, draw)
    assert abs(a - 32.5) < 2e-3
    # first step is the arithmetic midpoint of the range, and one iteration returns it
    assert modeling.binary_search_alpha(32.5, 1000, 3, 1, draw) == (1e-6 + 1e6) / 2
    # two iterations: the first midpoint is too uniform, so hi moves down
    assert modeling.binary_search_alpha(32.5, 1000, 3, 2, draw) == (1e-6 + (1e-6 + 1e6) / 2) / 2


def test_exemplar_is_sorted_unit_and_label_free():
    rng = np.random.default_rng(0)
    counts = [rng.integers(0, 50, 64) for _ in range(10)]
    ex = modeling.exemplar(counts)
    assert np.all(np.diff(ex) <= 1e-15)
    assert np.sum(ex * ex) == pytest.approx(1.0, rel=1e-12)
    ex2 = modeling.exemplar([rng.permutation(c) for c in counts])
    np.testing.assert_allclose(ex, ex2, rtol=1e-12)
    # one sample: the exemplar is just the normalised sorted vector
    one = modeling.exemplar([[3, 0, 4]])
    np.testing.assert_allclose(one, [0.8, 0.6, 0.0])
    assert modeling.exemplar_q30([[3, 0, 4]]).tolist() == [round(0.8 * 2 ** 30), round(0.6 * 2 ** 30), 0]


# ---- exponential and Beta families (paper Section V, the comparison of synthetic families) ----

def _geometric_eff(lam, E):
    # closed form of (sum r^i)^2 / sum r^(2i), r = exp(-lam)
    r = np.exp(-lam)
    if r == 1.0:
        return float(E)
    return ((1 - r ** E) / (1 - r)) ** 2 * (1 - r * r) / (1 - r ** (2 * E))


def test_exponential_family_closed_form_and_limits():
    for E in (8, 256):
        for lam in (0.0, 1e-3, 0.05, 0.7, 5.0):
            p = modeling.exponential_p(lam, E)
            assert abs(p.sum() - 1.0) < 1e-12 and np.all(np.diff(p) <= 0)
            assert np.isclose(modeling.eff_exp(p), _geometric_eff(lam, E), rtol=1e-10)
    assert np.isclose(modeling.eff_exp(modeling.exponential_p(0.0, 64)), 64.0)
    assert np.isclose(modeling.eff_exp(modeling.exponential_p(60.0, 64)), 1.0, rtol=1e-9)


def test_exponential_bisection_reaches_the_target_and_is_monotone():
    E = 256
    lams = []
    for X in (1.1, 1.5, 2.0, 4.0, 16.0):
        target = modeling.ddist_target(E, X)
        lam = modeling.binary_search_exponential(target, E)
        assert np.isclose(_geometric_eff(lam, E), target, rtol=1e-9)
        lams.append(lam)
    assert all(a < b for a, b in zip(lams, lams[1:]))   # a more skewed target needs a faster decay
    # large E, moderate decay: eff -> (1 + r) / (1 - r), i.e. lam = log((eff + 1) / (eff - 1))
    assert np.isclose(modeling.binary_search_exponential(20.0, 4096), np.log(21.0 / 19.0), rtol=1e-6)


def _beta_draw(seed):
    def draw(a, b, S, E):
        return np.random.default_rng(seed).beta(a, b, size=(S, E))
    return draw


def test_beta_family_law_of_large_numbers_and_grid_search():
    # iid x_i: eff_exp / E -> E[x]^2 / E[x^2] = a (a + b + 1) / ((a + 1) (a + b))
    E = 8192
    for a, b in ((0.5, 0.5), (2.0, 3.0), (0.2, 1.5)):
        p = modeling.beta_p(a, b, E, 4, _beta_draw(3))
        assert np.allclose(p.sum(axis=1), 1.0)
        got = np.mean([modeling.eff_exp(q) for q in p]) / E
        assert np.isclose(got, a * (a + b + 1) / ((a + 1) * (a + b)), rtol=0.03)
    # the brute-force search returns a grid point, and no other grid point is closer to the target
    E, S, target = 64, 8, 24.0
    a, b = modeling.grid_search_beta(target, E, S, _beta_draw(5), step=0.5, upper=2.0)
    assert a in (0.5, 1.0, 1.5, 2.0) and b in (0.5, 1.0, 1.5, 2.0)

    def mean_eff(a, b):
        p = modeling.beta_p(a, b, E, S, _beta_draw(5))
        return np.mean([modeling.eff_exp(q) for q in p])
    best = abs(mean_eff(a, b) - target)
    for aa in (0.5, 1.0, 1.5, 2.0):
        for bb in (0.5, 1.0, 1.5, 2.0):
            assert best <= abs(mean_eff(aa, bb) - target) + 1e-12


def test_families_matched_to_one_target_have_similar_sorted_shapes():
    # the paper compares the families by cosine similarity of sorted, L2-normalised vectors once they
    # are matched to the same eff_exp; matched vectors must be close to each other, far from uniform
    E, target = 256, 64.0
    lam = modeling.binary_search_exponential(target, E)
    pe = modeling.exponential_p(lam, E)
    rng = np.random.default_rng(0)
    alpha = (target - 1) / (E - target)           # closed-form Dirichlet inverse
    pd = rng.dirichlet(np.full(E, alpha))
    c = modeling.cosine(modeling.sorted_unit_vector(pe), modeling.sorted_unit_vector(pd))
    u = modeling.cosine(modeling.sorted_unit_vector(pe), modeling.sorted_unit_vector(np.ones(E)))
    assert c > 0.9 and c > u
    assert np.isclose(u, np.sqrt(target / E), rtol=1e-6)   # cosine to uniform = sqrt(eff_exp / E)
