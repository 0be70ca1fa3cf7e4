"""Pins of the router-selection oracle: library routines, closed forms and invariants."""
import numpy as np
import scipy.special

from oracle import router


def _logits(seed, T, E):
    return np.random.default_rng(seed).standard_normal((T, E)).astype(np.float32)


def test_ids_are_the_k_largest_in_descending_order_against_numpy_sort():
    z = _logits(1, 37, 53)
    ids, _ = router.topk_softmax(z, 6)
    order = np.argsort(-z.astype(np.float64), axis=1, kind="stable")[:, :6]
    assert np.array_equal(ids, order.astype(np.int32))
    picked = np.take_along_axis(z, ids.astype(np.int64), axis=1)
    assert np.all(np.diff(picked, axis=1) <= 0)
    rest_max = np.array([np.delete(z[t], ids[t]).max() for t in range(z.shape[0])])
    assert np.all(picked[:, -1] >= rest_max)


def test_k_equal_E_is_the_full_softmax():
    z = _logits(2, 9, 12)
    ids, w = router.topk_softmax(z, 12)
    ref = scipy.special.softmax(z.astype(np.float64), axis=1)
    for t in range(z.shape[0]):
        assert sorted(ids[t].tolist()) == list(range(12))
        assert np.allclose(w[t], ref[t][ids[t]], rtol=1e-6, atol=0)


def test_weights_closed_forms():
    # equal logits: every weight 1/k and the lowest indices are chosen in order
    ids, w = router.topk_softmax(np.zeros((3, 10), np.float32), 4)
    assert np.array_equal(ids, np.tile(np.arange(4, dtype=np.int32), (3, 1)))
    assert np.all(w == np.float32(0.25))
    # two selected logits a and b: weights are the logistic function of their difference
    z = np.full((1, 8), -50.0, np.float32)
    z[0, 5], z[0, 2] = 1.5, 0.25
    ids, w = router.topk_softmax(z, 2)
    assert ids.tolist() == [[5, 2]]
    assert np.allclose(w[0, 0], 1.0 / (1.0 + np.exp(-1.25)), rtol=1e-7)
    assert np.allclose(w.sum(), 1.0, rtol=1e-6)
    # k = 1: the argmax with weight exactly 1
    z = _logits(3, 20, 33)
    ids, w = router.topk_softmax(z, 1)
    assert np.array_equal(ids[:, 0], z.argmax(axis=1).astype(np.int32))
    assert np.all(w == 1.0)


def test_invariances():
    z = _logits(4, 11, 40)
    ids, w = router.topk_softmax(z, 5)
    # a constant added to a token's logits changes neither the choice nor (beyond rounding) the weights
    shift = np.float32(8.0)
    ids2, w2 = router.topk_softmax(z + shift, 5)
    assert np.array_equal(ids, ids2)
    assert np.allclose(w, w2, rtol=2e-6)
    # relabelling the experts relabels the ids and keeps the weights
    perm = np.random.default_rng(0).permutation(40)
    ids3, w3 = router.topk_softmax(z[:, perm], 5)
    assert np.array_equal(perm[ids3], ids)
    assert np.array_equal(w3, w)
    assert np.allclose(w.sum(axis=1), 1.0, rtol=1e-6)
    assert np.all(w > 0)


def test_ties_and_special_values():
    z = np.array([[1.0, 3.0, 3.0, 2.0, 3.0, -np.inf, np.nan, 0.5]], np.float32)
    ids, w = router.topk_softmax(z, 4)
    assert ids.tolist() == [[1, 2, 4, 3]]           # equal logits: lower index first
    e = np.exp(-1.0)
    assert np.allclose(w[0], np.array([1, 1, 1, e]) / (3 + e), rtol=1e-6)
    ids, w = router.topk_softmax(z, 8)
    assert ids[0, -1] == 6 and ids[0, -2] == 5       # -inf before NaN, NaN last
    assert w[0, -1] == 0 and w[0, -2] == 0
