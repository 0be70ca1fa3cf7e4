"""Pins for the integer half of the oracle: closed forms of Effective Experts
(Section III-A, Eq. 2), invariants of histogram / offsets / permutation, the
padded-tile formula, and the selector's defining properties (Section IV)."""
import itertools

import numpy as np
import pytest

import damoe_inputs as di
from oracle import modeling, route


# ---- Effective Experts ------------------------------------------------------

def test_eff_exp_uniform_is_E():
    for E in (8, 256, 384):
        _, _, v = route.effective_experts([7] * E)
        assert v == float(E)


def test_eff_exp_single_expert_is_one():
    h = [0] * 256
    h[17] = 4096
    assert route.effective_experts(h)[2] == 1.0


def test_eff_exp_same_k_experts_for_all_tokens_is_k():
    ids = np.tile(np.array([[3, 9, 27, 81, 100, 5, 6, 7]], dtype=np.int32), (64, 1))
    assert route.effective_experts(route.histogram(ids, 256))[2] == 8.0


def test_eff_exp_m_equal_experts_is_m():
    for m in (1, 2, 5, 100):
        h = [13] * m + [0] * (256 - m)
        assert route.effective_experts(h)[2] == float(m)


def test_eff_exp_hand_value():
    # counts (3,1): (3+1)^2 / (9+1) = 1.6
    assert route.effective_experts([3, 1])[2] == 1.6
    assert route.effective_experts([3, 1])[:2] == (4, 10)


def test_eff_exp_scale_and_relabel_invariant_and_range():
    rng = np.random.default_rng(0)
    for _ in range(50):
        h = rng.integers(0, 200, size=64)
        if h.sum() == 0:
            continue
        v = route.effective_experts(h)[2]
        assert 1.0 <= v <= 64.0
        assert route.effective_experts(h * 7)[2] == pytest.approx(v, rel=1e-15)
        assert route.effective_experts(rng.permutation(h))[2] == v
        # same statistic through the fp64 formula on fractions
        assert modeling.eff_exp(h / h.sum()) == pytest.approx(v, rel=1e-12)


def test_eff_exp_no_valid_id():
    assert route.effective_experts([0, 0, 0]) == (0, 0, 0.0)


# ---- histogram / offsets / permutation ---------------------------------------

def test_histogram_brute_force_and_sum():
    ids, _, _ = di.routing_batch(0, 64, 2, 8, 1.0)
    h = route.histogram(ids, 8)
    want = [sum(1 for t in range(64) for j in range(2) if ids[t, j] == e) for e in range(8)]
    assert h.tolist() == want
    assert h.sum() == 64 * 2
    assert h.max() <= 64            # distinct experts per token


def test_histogram_matches_bincount_library():
    ids, _, _ = di.routing_batch(3, 1024, 8, 256, 0.2)
    assert np.array_equal(route.histogram(ids, 256), np.bincount(ids.reshape(-1), minlength=256))


def test_invalid_ids_are_skipped():
    ids = np.array([[0, 5], [-1, 1], [8, 0]], dtype=np.int32)
    h = route.histogram(ids, 8)
    assert h.tolist() == [2, 1, 0, 0, 0, 1, 0, 0]
    off, perm, inv = route.offsets_and_permutation(ids, 8)
    assert off[-1] == 4 and len(perm) == 4
    assert inv.tolist() == [0, 3, -1, 2, -1, 1]


def test_permutation_invariants():
    for seed, (T, k, E, a) in enumerate([(64, 2, 8, 1.0), (64, 8, 256, 0.05), (300, 8, 384, 10.0), (1, 8, 256, 1.0)]):
        ids, _, _ = di.routing_batch(seed, T, k, E, a)
        flat = ids.reshape(-1)
        off, perm, inv = route.offsets_and_permutation(ids, E)
        P = T * k
        assert off[0] == 0 and off[E] == P and np.all(np.diff(off) >= 0)
        assert sorted(perm.tolist()) == list(range(P))             # bijection
        assert np.array_equal(inv[perm], np.arange(P))
        for e in range(E):
            seg = perm[off[e]:off[e + 1]]
            assert np.all(flat[seg] == e)
            assert np.all(np.diff(seg) > 0)                        # stable: ascending flat index
        # the same grouping through a library stable sort
        assert np.array_equal(perm, np.argsort(flat, kind="stable"))


def test_duplicates_within_a_token_are_legal():
    ids = np.array([[2, 2], [2, 1]], dtype=np.int32)
    off, perm, inv = route.offsets_and_permutation(ids, 4)
    assert off.tolist() == [0, 0, 1, 4, 4]
    assert perm.tolist() == [3, 0, 1, 2]


# ---- tile counts --------------------------------------------------------------

def test_tile_counts_formula_and_bounds():
    ids, _, _ = di.routing_batch(1, 256, 8, 256, 0.05)
    h = route.histogram(ids, 256)
    P, A = int(h.sum()), route.active_experts(h)
    ns = [1, 8, 16, 32, 64, 128, 256, 100000]
    tiles = route.tile_counts(h, ns)
    assert tiles[0] == P and tiles[-1] == A
    assert np.all(np.diff(tiles) <= 0)
    for n, t in zip(ns, tiles):
        assert t == sum(int(np.ceil(x / n)) for x in h)
        assert -(-P // n) <= t <= A + (P - A) // n
    pref = route.tile_prefix(h, 32)
    assert pref[-1] == tiles[3] and pref[0] == 0


def test_tile_counts_tiny_by_hand():
    # counts 0, 1, 8, 9, 17 with N = 8 -> 0 + 1 + 1 + 2 + 3
    assert route.tile_counts([0, 1, 8, 9, 17], [8])[0] == 7


# ---- selector -------------------------------------------------------------------

def test_pick_bucket():
    b = [1, 4, 16, 64, 256]
    assert route.pick_bucket(b, 1) == 0
    assert route.pick_bucket(b, 5) == 2
    assert route.pick_bucket(b, 64) == 3
    assert route.pick_bucket(b, 9999) == 4
    assert route.pick_bucket([64, 16, 256], 17) == 0


def _exemplars_for(E, k, T, alphas, seed0=100, S=4):
    out = []
    for i, a in enumerate(alphas):
        counts = [route.histogram(di.routing_batch(seed0 + 10 * i + s, T, k, E, a)[0], E) for s in range(S)]
        out.append(modeling.exemplar_q30(counts))
    return out


def test_own_exemplar_wins():
    # an exemplar built from the query itself has cosine 1 and must win (Cauchy-Schwarz)
    E, k, T = 256, 8, 64
    ex = _exemplars_for(E, k, T, [0.05, 0.2, 1.0, 10.0])
    h = route.histogram(di.routing_batch(999, T, k, E, 0.5)[0], E)
    ex.append(modeling.exemplar_q30([h]))
    ids = [10, 11, 12, 13, 77]
    assert route.select_exemplar(h, ex, ids) == 77


def test_selection_ignores_expert_labels_and_scale():
    E, k, T = 256, 8, 64
    ex = _exemplars_for(E, k, T, [0.05, 0.2, 1.0, 10.0])
    vids = [0, 1, 2, 3]
    rng = np.random.default_rng(5)
    for s in range(8):
        h = route.histogram(di.routing_batch(500 + s, T, k, E, [0.05, 0.3, 2.0, 8.0][s % 4])[0], E)
        v = route.select_exemplar(h, ex, vids)
        assert route.select_exemplar(rng.permutation(h), ex, vids) == v
        assert route.select_exemplar(h * 3, ex, vids) == v


def test_selection_agrees_with_float_cosine_when_margin_is_clear():
    E, k, T = 256, 8, 256
    alphas = [0.05, 0.2, 1.0, 10.0]
    ex = _exemplars_for(E, k, T, alphas)
    for s in range(12):
        h = route.histogram(di.routing_batch(700 + s, T, k, E, alphas[s % 4])[0], E)
        cos = [modeling.cosine(np.sort(h)[::-1], e.astype(np.float64)) for e in ex]
        order = np.argsort(cos)
        if cos[order[-1]] - cos[order[-2]] > 2.0 ** -20:
            assert route.select_exemplar(h, ex, list(range(4))) == int(order[-1])
    # skewed queries pick the skewed exemplar, uniform queries the uniform one
    h_skew = route.histogram(di.routing_batch(1, T, k, E, 0.05)[0], E)
    h_unif = route.histogram(di.routing_batch(2, T, k, E, 10.0)[0], E)
    assert route.select_exemplar(h_skew, ex, list(range(4))) == 0
    assert route.select_exemplar(h_unif, ex, list(range(4))) == 3


def test_exemplar_tie_goes_to_lowest_index():
    h = [4, 3, 2, 1]
    e = modeling.exemplar_q30([h])
    assert route.select_exemplar(h, [e, e.copy()], [5, 6]) == 5


def test_effexp_bins():
    den = 1 << 16
    th = [int(2.0 * den), int(3.5 * den)]       # bins: <2, [2,3.5), >=3.5
    var = [7, 8, 9]
    assert route.select_effexp_bins([10, 0, 0, 0], th, den, var) == 7      # eff 1
    assert route.select_effexp_bins([5, 5, 0, 0], th, den, var) == 8       # eff 2 (boundary belongs above)
    assert route.select_effexp_bins([5, 5, 5, 0], th, den, var) == 8       # eff 3
    assert route.select_effexp_bins([5, 5, 5, 5], th, den, var) == 9       # eff 4


def test_cost_selector_brute_force():
    rng = np.random.default_rng(3)
    ns = [16, 32, 64, 128, 256]
    for s in range(20):
        h = route.histogram(di.routing_batch(s, int(rng.integers(1, 600)), 8, 256, float(rng.choice([0.05, 1, 10])))[0], 256)
        cf = rng.integers(0, 10 ** 6, 5)
        cb = rng.integers(1, 10 ** 7, 5)
        cr = rng.integers(1, 10 ** 6, 5)
        cl = rng.integers(1, 10 ** 5, 5)
        A = int((h > 0).sum())
        costs = []
        for v, n in enumerate(ns):
            tiles = sum((int(x) + n - 1) // n for x in h)
            costs.append(int(cf[v]) + max(int(cb[v]) * A + int(cr[v]) * (tiles - A), int(cl[v]) * tiles * n))
        assert route.variant_costs(h, ns, cf, cb, cr, cl) == costs
        assert route.select_cost(h, ns, cf, cb, cr, cl) == int(np.argmin(costs))


def test_select_variant_dispatch_and_static():
    E = 8
    h = [9, 3, 1, 0, 0, 0, 0, 3]
    ex_a = modeling.exemplar_q30([[16, 0, 0, 0, 0, 0, 0, 0]])
    ex_b = modeling.exemplar_q30([[2] * 8])
    bucket = dict(T=64, static_variant=4, exemplars=[ex_a, ex_b], exemplar_variants=[1, 2],
                  bin_thresholds_num=[3 << 16], bin_den=1 << 16, bin_variants=[5, 6],
                  c_fix=[0, 0], c_byte=[10, 10], c_reload=[1, 1], c_flop=[1, 100])
    small = dict(bucket, T=16, static_variant=0)
    for mode, want in ((route.MODE_EXEMPLAR, 1), (route.MODE_EFFEXP_BINS, 5), (route.MODE_COST, 0)):
        table = dict(mode=mode, buckets=[small, bucket])
        assert route.select_variant(table, h, 40, [8, 16]) == want
        assert route.select_variant(table, h, 40, [8, 16], static=True) == 4
        assert route.select_variant(table, h, 3, [8, 16], static=True) == 0
