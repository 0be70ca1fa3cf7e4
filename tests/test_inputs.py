"""The seeded input generators: determinism, device independence of the integer
hash, and the statistics the Dirichlet routing model must have (Section II-D)."""
import numpy as np
import torch

import damoe_inputs as di


def test_mix64_matches_python_ints():
    def mix(z):
        z &= (1 << 64) - 1
        z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & ((1 << 64) - 1)
        z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & ((1 << 64) - 1)
        return z ^ (z >> 31)
    vals = [0, 1, 2, 12345678901234567, (1 << 63) + 5, (1 << 64) - 1]
    t = torch.tensor([di._wrap64(v) for v in vals], dtype=torch.int64)
    got = di._mix64(t).tolist()
    assert [g & ((1 << 64) - 1) for g in got] == [mix(v) for v in vals]


def test_normal_bf16_is_counter_based():
    a = di.normal_bf16(3, di.TID_W13, 0, 4096, 0.02)
    b = di.normal_bf16(3, di.TID_W13, 1024, 1024, 0.02)
    assert torch.equal(a[1024:2048].view(torch.int16), b.view(torch.int16))
    c = di.normal_bf16(4, di.TID_W13, 0, 4096, 0.02)
    assert not torch.equal(a.view(torch.int16), c.view(torch.int16))


def test_normal_bf16_moments():
    a = di.normal_bf16(0, di.TID_X, 0, 1 << 20, 1.0).double()
    assert abs(a.mean().item()) < 5e-3
    assert abs(a.std().item() - 1.0) < 5e-3
    w = di.normal_bf16(0, di.TID_W2, 0, 1 << 20, 0.02).double()
    assert abs(w.std().item() - 0.02) < 2e-4


def test_expert_slices_agree_with_materialized():
    W = di.MoEWeights(5, 3, 128, 128)
    w13, w2 = W.materialize("cpu")
    assert torch.equal(w13[2].view(torch.int16), W.expert_w13(2).view(torch.int16))
    assert torch.equal(w2[1].view(torch.int16), W.expert_w2(1).view(torch.int16))


def test_dirichlet_simplex_and_moments():
    E = 256
    for alpha in (0.05, 1.0, 10.0):
        p = di.dirichlet_p(alpha, E, 400, di._rng(1, 0))
        assert np.all(p >= 0)
        np.testing.assert_allclose(p.sum(axis=1), 1.0, rtol=1e-12)
        # E[sum p^2] = (alpha + 1) / (E alpha + 1) for the symmetric Dirichlet
        want = (alpha + 1) / (E * alpha + 1)
        got = (p ** 2).sum(axis=1).mean()
        assert abs(got - want) / want < 0.08
        # marginal mean 1/E
        assert abs(p.mean() - 1 / E) < 1e-12 + 1e-9


def test_dirichlet_tiny_alpha_does_not_underflow():
    p = di.dirichlet_p(1e-6, 64, 16, di._rng(2, 0))
    assert np.all(np.isfinite(p))
    np.testing.assert_allclose(p.sum(axis=1), 1.0, rtol=1e-12)
    assert np.all(p.max(axis=1) > 0.99)


def test_routing_distinct_and_proportional():
    ids, w, p = di.routing_batch(0, 4096, 2, 8, 1.0)
    assert ids.shape == (4096, 2) and ids.dtype == np.int32
    assert np.all(ids[:, 0] != ids[:, 1])
    assert np.all((ids >= 0) & (ids < 8))
    # first draw is a plain categorical draw from p
    freq = np.bincount(ids[:, 0], minlength=8) / 4096.0
    assert np.abs(freq - p).max() < 0.03
    np.testing.assert_allclose(w.sum(axis=1), 1.0, rtol=1e-6)
    assert w.dtype == np.float32


def test_routing_is_seeded():
    a = di.routing_batch(7, 64, 8, 256, 0.2)
    b = di.routing_batch(7, 64, 8, 256, 0.2)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])
    c = di.routing_batch(8, 64, 8, 256, 0.2)
    assert not np.array_equal(a[0], c[0])


def test_trace_batches_range():
    tr = di.trace_batches(1000, 500)
    assert len(tr) == 500
    assert all(1 <= T <= 4096 and 0.05 <= a <= 10.0 for T, a in tr)
    assert min(T for T, _ in tr) <= 4 and max(T for T, _ in tr) >= 2048
