"""Router selection on the GPU against the oracle: ids bit for bit, weights within float32
rounding (expf within an ulp, a sum of at most 32 terms, one correctly rounded division), and the
layer call that starts from logits against the layer call that is given the same ids and weights."""
import numpy as np
import pytest
import torch

import damoe_inputs as di
from helpers import Case, bits16, config0, max_scaled_err, rel_frobenius
from oracle import codecs, layer, router

pytestmark = pytest.mark.gpu

W_RTOL = 2e-6


@pytest.fixture(scope="module")
def d():
    import paper_2607_23099_b200 as d
    return d


@pytest.mark.parametrize("T,E,k,alpha", [(64, 8, 2, 1.0), (333, 256, 8, 0.2), (1, 384, 8, 1.0), (2048, 256, 8, 10.0),
                                         (17, 1000, 32, 0.05), (5, 32, 32, 1.0)])
def test_router_topk_matches_oracle(d, T, E, k, alpha):
    z = di.router_logits(11 + T, T, E, alpha)
    if T >= 5:  # rows with ties, infinities and a NaN
        z[1, :] = 0.0
        z[2, : E // 2] = z[2, E // 2]
        z[3, 0] = -np.inf
        z[3, E - 1] = np.inf
        z[4, E // 3] = np.nan
    m = d.DAMoE(max(T, 1), k, E, 128, 128)
    ids, w = m.router_topk(torch.from_numpy(z).cuda())
    torch.cuda.synchronize()
    ref_ids, ref_w = router.topk_softmax(z, k)
    assert np.array_equal(ids.cpu().numpy(), ref_ids)
    got_w = w.cpu().numpy()
    finite = np.isfinite(ref_w)
    assert np.array_equal(np.isfinite(got_w), finite)
    assert np.allclose(got_w[finite], ref_w[finite], rtol=W_RTOL, atol=1e-12)
    m.close()


def test_layer_from_logits(d):
    case = config0(seed=5, T=64)
    dev = "cuda:0"
    w13, w2 = case.weights.materialize(dev)
    z = di.router_logits(77, case.T, case.E, 0.5)
    z_d = torch.from_numpy(z).to(dev)
    m = d.DAMoE(64, case.k, case.E, case.H, case.I)
    x = case.x(dev)
    out = m.moe_from_logits(x, w13, w2, z_d, d.VARIANT_AUTO)
    sel_ids, sel_w = m.debug_fetch_routing(case.T)
    ref_ids, ref_w = router.topk_softmax(z, case.k)
    assert np.array_equal(sel_ids, ref_ids)
    assert np.allclose(sel_w, ref_w, rtol=W_RTOL)
    # the same layer given the selected ids and weights explicitly: identical bits
    ids_d, w_d = m.router_topk(z_d)
    out2 = m.fused_moe(x, w13, w2, ids_d, w_d, d.VARIANT_AUTO)
    assert torch.equal(out.view(torch.int16), out2.view(torch.int16))
    # and the oracle's layer on the oracle's routing
    ref_bits, _ = layer.moe_layer_bf16(bits16(case.x()), case.w13_bits, case.w2_bits, ref_ids, ref_w, case.E)
    got, ref = codecs.bf16_decode(bits16(out)), codecs.bf16_decode(ref_bits)
    assert rel_frobenius(got, ref) <= 5e-3
    assert max_scaled_err(got, ref) <= 1e-2
    assert m.debug_fetch(case.T)["status"] == 0
    # an empty batch is a no-op
    m.moe_from_logits(x[:0], w13, w2, z_d[:0], d.VARIANT_AUTO)
    m.close()
