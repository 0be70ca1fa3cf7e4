"""Host logic of the offline auto-tuner (no GPU): the product's exemplar builder against the
oracle's, bucket construction from sweep rows, and the byte layout it feeds to the library."""
import numpy as np

import damoe_inputs as di
from oracle import modeling, route


def _autotune():
    import __graft_entry__ as g
    g.load_build_module().build()
    from paper_2607_23099_b200 import autotune
    return autotune


def test_exemplar_builder_matches_oracle():
    at = _autotune()
    for seed, (T, E, a) in enumerate([(64, 256, 0.05), (256, 256, 1.0), (1024, 384, 10.0), (1, 256, 1.0)]):
        counts = [np.bincount(di.routing_batch(seed * 10 + s, T, 8, E, a)[0].reshape(-1), minlength=E) for s in range(4)]
        assert at.exemplar_q30(counts) == modeling.exemplar_q30(counts).tolist()
        assert abs(at.effective_experts(counts[0]) - route.effective_experts(counts[0])[2]) < 1e-9


def test_build_bucket_picks_fastest_and_static_from_uniform():
    at = _autotune()
    ns, V, E = [16, 32, 64, 128, 256], 5, 32
    rng = np.random.default_rng(0)

    def cell(alpha, best):
        us = [[100.0 + 10 * abs(v - best) for v in range(V)] for _ in range(2)]
        counts = [rng.integers(0, 9, E).tolist() for _ in range(2)]
        return dict(alpha=alpha, counts=counts, us=us, active=[20, 21], tiles=[[30, 25, 22, 21, 20], [31, 26, 23, 22, 21]])

    b = at.build_bucket(64, [cell(0.05, 3), cell(1.0, 1), cell(at.UNIFORM, 0)], ns, V)
    assert b["static_variant"] == 0 and b["exemplar_variants"] == [3, 1]
    assert len(b["exemplars"]) == 2 and len(b["exemplars"][0]) == E
    assert len(b["bin_variants"]) == len(b["bin_thresholds_num"]) + 1
    assert all(len(b[k]) == V and min(b[k]) >= 0 for k in ("c_fix", "c_byte", "c_reload", "c_flop"))
    from paper_2607_23099_b200 import tuning
    blob = tuning.pack_table(dict(mode=0, buckets=[b]), E, 8, 1024, 512, 0, V)
    assert blob[:8] == b"DAMOETB1" and len(blob) > 44 + 2 * 4 * E
