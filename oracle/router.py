"""Router selection, the step upstream of the expert layer, written the slow and obvious way.

TEST INFRASTRUCTURE ONLY.  Nothing on the product path may import this module;
it shares no code with the CUDA library.

What the paper fixes
  * the end-to-end MoE-layer latency it reports covers "router selection,
    routing-metadata construction, dispatch and fused-MoE execution" (Section V), and the
    histogram is built from the router's top-k choice (Fig. 9(b), step 5).

Readings taken where the paper is silent (listed in the design notes)
  * per token the k experts with the largest logits are selected; among equal logits the lower
    expert index comes first; NaN sorts below every number;
  * the routing weights are the softmax over the k selected logits (the gating of the
    build's configurations), computed here in float64 and rounded once to float32;
  * ids are stored in order of descending logit.
"""
from __future__ import annotations

import math

import numpy as np


def topk_softmax(logits, k: int):
    """(topk_ids [T, k] int32, topk_weights [T, k] float32) from logits [T, E] float32."""
    z = np.asarray(logits, dtype=np.float32)
    T, E = z.shape
    assert 1 <= k <= E
    ids = np.zeros((T, k), dtype=np.int32)
    w = np.zeros((T, k), dtype=np.float32)
    for t in range(T):
        row = [float(v) for v in z[t]]
        left = list(range(E))
        chosen = []
        for _ in range(k):
            best = None
            for e in left:  # a plain scan: larger value wins, NaN never beats a number, first index wins ties
                if best is None:
                    best = e
                    continue
                a, b = row[e], row[best]
                if math.isnan(b) and not math.isnan(a):
                    best = e
                elif not math.isnan(a) and not math.isnan(b) and a > b:
                    best = e
            chosen.append(best)
            left.remove(best)
        top = row[chosen[0]]
        ex = [0.0 if math.isnan(row[e]) else math.exp(row[e] - top) for e in chosen]
        s = sum(ex)
        ids[t] = chosen
        w[t] = [np.float32(v / s) if s > 0 else np.float32(float("nan")) for v in ex]
    return ids, w
