"""The fused-MoE expert layer in fp64.

TEST INFRASTRUCTURE ONLY.  Nothing on the product path may import this module;
it shares no code with the CUDA library.

The paper treats the expert computation as per-expert GEMMs C = A x B with A the
expert's weight matrix and B the tokens routed to it (Fig. 3, Section II-C) and
says nothing more about the FFN.  The reading taken here is the usual gated FFN
of the models it serves:

    for every token t and slot j < k, with e = ids[t, j]:
        g = W13[e, 0:I , :] . x_t          (gate projection)
        u = W13[e, I:2I, :] . x_t          (up projection)
        a = g / (1 + exp(-g)) * u          (SwiGLU)
        h = bf16(a)                        (the one inner rounding point)
        y = W2[e] . h
    out_t = bf16( sum_j w[t, j] * y_(t,j) ),   j ascending

All arithmetic is binary64 on the exactly decoded bf16 / E4M3 inputs.  An id
outside [0, E) contributes nothing.  Weights may be given as arrays or as
callables e -> array so that one expert at a time is held in memory.
"""
from __future__ import annotations

import numpy as np

from .codecs import bf16_decode, bf16_rne, bf16_round, e4m3_decode, e4m3_rne_sat


def _get(w, e):
    return w(e) if callable(w) else w[e]


def swiglu(g, u):
    return g / (1.0 + np.exp(-g)) * u


def moe_layer_bf16(x_bits, w13_bits, w2_bits, topk_ids, topk_weights, E: int, tokens=None):
    """x_bits [T,H] uint16; w13_bits [E,2I,H] / w2_bits [E,H,I] uint16 arrays or
    callables; topk_ids [T,k]; topk_weights [T,k] float32.

    Returns (out_bits [n,H] uint16, out64 [n,H] float64 before the final rounding)
    for the tokens listed in ``tokens`` (all tokens when None).
    """
    x_bits = np.asarray(x_bits)
    ids = np.asarray(topk_ids)
    wts = np.asarray(topk_weights, dtype=np.float32).astype(np.float64)
    T, H = x_bits.shape
    k = ids.shape[1]
    tok = np.arange(T) if tokens is None else np.asarray(tokens)
    x = bf16_decode(x_bits[tok])                                   # [n, H]
    y = np.zeros((len(tok), k, H), dtype=np.float64)
    for e in sorted(set(int(v) for v in ids[tok].reshape(-1) if 0 <= v < E)):
        rows, slots = np.nonzero(ids[tok] == e)
        w13 = bf16_decode(_get(w13_bits, e))                       # [2I, H]
        I = w13.shape[0] // 2
        xe = x[rows]                                               # [m, H]
        g = xe @ w13[:I].T
        u = xe @ w13[I:].T
        h = bf16_round(swiglu(g, u))                               # [m, I]
        del w13
        w2 = bf16_decode(_get(w2_bits, e))                         # [H, I]
        y[rows, slots] = h @ w2.T
        del w2
    out64 = np.zeros((len(tok), H), dtype=np.float64)
    for j in range(k):
        valid = ((ids[tok, j] >= 0) & (ids[tok, j] < E)).astype(np.float64)
        out64 += (wts[tok, j] * valid)[:, None] * y[:, j]
    return bf16_rne(out64), out64


def quantize_act_e4m3(h_b):
    """Per (row, group of 128 consecutive channels) re-quantisation of a bf16
    activation to E4M3 with an fp32 scale: s = amax/448 (1 when amax == 0),
    code = e4m3(fp32(h)/s), both steps in binary32."""
    h32 = np.asarray(h_b, dtype=np.float64).astype(np.float32)
    m, I = h32.shape
    grp = h32.reshape(m, I // 128, 128)
    amax = np.abs(grp).max(axis=2)
    s = np.where(amax == 0, np.float32(1.0), amax / np.float32(448.0)).astype(np.float32)
    scaled = (grp / s[:, :, None]).astype(np.float32)
    codes = e4m3_rne_sat(scaled.astype(np.float64)).reshape(m, I)
    return codes, s


def moe_layer_fp8(xq, x_scale, w13q, w13_scale, w2q, w2_scale, topk_ids, topk_weights, E: int,
                  tokens=None):
    """Block-scaled FP8 layer.  xq [T,H] uint8 codes with x_scale [T,H/128] fp32;
    w13q [E,2I,H] with w13_scale [E,2I/128,H/128]; w2q [E,H,I] with w2_scale
    [E,H/128,I/128] (arrays or callables per expert).  The activation h is
    rounded to bf16 and then re-quantised per 1x128 group (quantize_act_e4m3)."""
    xq = np.asarray(xq)
    ids = np.asarray(topk_ids)
    wts = np.asarray(topk_weights, dtype=np.float32).astype(np.float64)
    T, H = xq.shape
    k = ids.shape[1]
    tok = np.arange(T) if tokens is None else np.asarray(tokens)
    xs = np.asarray(x_scale, dtype=np.float32).astype(np.float64)
    x = e4m3_decode(xq[tok]) * np.repeat(xs[tok], 128, axis=1)
    y = np.zeros((len(tok), k, H), dtype=np.float64)
    for e in sorted(set(int(v) for v in ids[tok].reshape(-1) if 0 <= v < E)):
        rows, slots = np.nonzero(ids[tok] == e)
        s13 = np.asarray(_get(w13_scale, e), dtype=np.float32).astype(np.float64)
        w13 = e4m3_decode(_get(w13q, e)) * np.repeat(np.repeat(s13, 128, axis=0), 128, axis=1)
        I = w13.shape[0] // 2
        xe = x[rows]
        g = xe @ w13[:I].T
        u = xe @ w13[I:].T
        h_b = bf16_round(swiglu(g, u))
        hq, hs = quantize_act_e4m3(h_b)
        h_hat = e4m3_decode(hq) * np.repeat(hs.astype(np.float64), 128, axis=1)
        s2 = np.asarray(_get(w2_scale, e), dtype=np.float32).astype(np.float64)
        w2 = e4m3_decode(_get(w2q, e)) * np.repeat(np.repeat(s2, 128, axis=0), 128, axis=1)
        y[rows, slots] = h_hat @ w2.T
    out64 = np.zeros((len(tok), H), dtype=np.float64)
    for j in range(k):
        valid = ((ids[tok, j] >= 0) & (ids[tok, j] < E)).astype(np.float64)
        out64 += (wts[tok, j] * valid)[:, None] * y[:, j]
    return bf16_rne(out64), out64
