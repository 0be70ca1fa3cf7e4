"""Routing statistics, permutation, tile counts and kernel selection: the integer
half of the distribution-aware fused-MoE path, written the slow and obvious way.

TEST INFRASTRUCTURE ONLY.  Nothing on the product path may import this module;
it shares no code with the CUDA library.

What the paper fixes
  * t_i, the number of tokens routed to expert i in one forward pass, and the
    Effective Experts statistic (sum t_i)^2 / sum t_i^2          (Section III-A, Eq. 2)
  * expert GEMMs pad each expert's token columns up to the tile width N, so a
    kernel with tile width N runs sum_i ceil(t_i / N) token tiles  (Fig. 3, Section II-C)
  * the online dispatcher sorts the histogram in descending order and takes the
    exemplar of the current token-count bucket with the highest cosine
    similarity, one dot product per unit-norm exemplar           (Section IV-A, IV-B)
  * the comparison baseline keeps one statically chosen kernel per token-count
    bucket                                                        (Section IV, Section V)

Readings taken where the paper is silent (all listed in the design notes)
  * the histogram is built from the top-k expert ids; an id outside [0, E) is
    skipped;
  * the canonical order of (token, slot) pairs inside an expert's segment is
    ascending flat index p = t*k + j (a stable counting sort);
  * the bucket of a token count T is the smallest bucket >= T, else the largest;
  * exemplars are stored as round(e_i * 2^30) and scored in exact integer
    arithmetic; ties go to the lowest index;
  * besides exemplar matching, a table may select by Effective-Experts bins or
    by an integer cost model over padded tiles and weight reloads.
"""
from __future__ import annotations

import numpy as np

MODE_EXEMPLAR, MODE_EFFEXP_BINS, MODE_COST = 0, 1, 2


def histogram(topk_ids, E: int) -> np.ndarray:
    """t_i of Eq. 2: how many (token, slot) pairs name expert i."""
    hist = np.zeros(E, dtype=np.int64)
    for e in np.asarray(topk_ids).reshape(-1):
        if 0 <= e < E:
            hist[e] += 1
    return hist


def effective_experts(hist):
    """Eq. 2.  Returns (sum1, sum2, eff_exp) with the sums as Python ints and the
    ratio as one binary64 division; 0.0 when no valid id exists."""
    sum1 = sum(int(t) for t in hist)
    sum2 = sum(int(t) * int(t) for t in hist)
    if sum2 == 0:
        return sum1, sum2, 0.0
    return sum1, sum2, float(sum1 * sum1) / float(sum2)


def offsets_and_permutation(topk_ids, E: int):
    """Exclusive scan of the histogram and the stable grouping of pairs by expert.

    perm[q] = flat pair index p = t*k + j sitting at sorted position q;
    inv[p]  = q, or -1 for a pair whose id is out of range.
    """
    ids = np.asarray(topk_ids).reshape(-1)
    hist = histogram(ids, E)
    offsets = np.zeros(E + 1, dtype=np.int64)
    for e in range(E):
        offsets[e + 1] = offsets[e] + hist[e]
    cursor = offsets[:-1].copy()
    perm = np.full(int(offsets[E]), -1, dtype=np.int64)
    inv = np.full(ids.shape[0], -1, dtype=np.int64)
    for p, e in enumerate(ids):
        if 0 <= e < E:
            q = cursor[e]
            cursor[e] += 1
            perm[q] = p
            inv[p] = q
    return offsets, perm, inv


def tile_counts(hist, tile_ns):
    """Token tiles each tile width needs: sum_e ceil(t_e / N)."""
    return np.array([sum(-(-int(t) // int(n)) for t in hist) for n in tile_ns], dtype=np.int64)


def tile_prefix(hist, n: int) -> np.ndarray:
    """Exclusive scan of ceil(t_e / n): where each expert's token tiles start."""
    out = np.zeros(len(hist) + 1, dtype=np.int64)
    for e, t in enumerate(hist):
        out[e + 1] = out[e] + (-(-int(t) // n))
    return out


def active_experts(hist) -> int:
    return int(sum(1 for t in hist if t > 0))


def pick_bucket(bucket_Ts, T: int) -> int:
    """Index of the smallest bucket >= T, else of the largest bucket."""
    best = None
    for i, b in enumerate(bucket_Ts):
        if b >= T and (best is None or b < bucket_Ts[best]):
            best = i
    if best is None:
        best = max(range(len(bucket_Ts)), key=lambda i: bucket_Ts[i])
    return best


def exemplar_scores(hist, exemplars_q30):
    """Dot product of the descending-sorted histogram with every fixed-point
    exemplar (Section IV-B); exact integers."""
    q = sorted((int(t) for t in hist), reverse=True)
    return [sum(qi * int(ei) for qi, ei in zip(q, ex)) for ex in exemplars_q30]


def select_exemplar(hist, exemplars_q30, kernel_ids):
    scores = exemplar_scores(hist, exemplars_q30)
    best = 0
    for m in range(1, len(scores)):
        if scores[m] > scores[best]:
            best = m
    return int(kernel_ids[best])


def select_effexp_bins(hist, thresholds_num, den: int, bin_variants):
    """bin r holds eff_exp in [theta_{r-1}, theta_r), theta = num/den; the
    comparison sum1^2 * den >= num * sum2 is exact."""
    sum1, sum2, _ = effective_experts(hist)
    r = 0
    for num in thresholds_num:
        if sum1 * sum1 * int(den) >= int(num) * sum2:
            r += 1
    return int(bin_variants[r])


def variant_costs(hist, tile_ns, c_fix, c_byte, c_reload, c_flop):
    """cost_v = c_fix + max(c_byte*A + c_reload*(tiles_v - A), c_flop*tiles_v*N_v)."""
    A = active_experts(hist)
    tiles = tile_counts(hist, tile_ns)
    costs = []
    for v, n in enumerate(tile_ns):
        mem = int(c_byte[v]) * A + int(c_reload[v]) * (int(tiles[v]) - A)
        mma = int(c_flop[v]) * int(tiles[v]) * int(n)
        costs.append(int(c_fix[v]) + max(mem, mma))
    return costs


def select_cost(hist, tile_ns, c_fix, c_byte, c_reload, c_flop, enabled=None):
    costs = variant_costs(hist, tile_ns, c_fix, c_byte, c_reload, c_flop)
    best = None
    for v, c in enumerate(costs):
        if enabled is not None and not enabled[v]:
            continue
        if best is None or c < costs[best]:
            best = v
    return int(best)


def select_variant(table: dict, hist, T: int, tile_ns, static: bool = False) -> int:
    """The dispatcher: pick the bucket from T, then apply the table's mode.

    ``table`` = {"mode": m, "buckets": [{"T":..., "static_variant":...,
      "exemplars": [[q30]*E, ...], "exemplar_variants": [...],
      "bin_thresholds_num": [...], "bin_den": d, "bin_variants": [...],
      "c_fix": [...], "c_byte": [...], "c_reload": [...], "c_flop": [...]}, ...]}
    """
    b = table["buckets"][pick_bucket([bk["T"] for bk in table["buckets"]], T)]
    if static:
        return int(b["static_variant"])
    mode = table["mode"]
    if mode == MODE_EXEMPLAR:
        return select_exemplar(hist, b["exemplars"], b["exemplar_variants"])
    if mode == MODE_EFFEXP_BINS:
        return select_effexp_bins(hist, b["bin_thresholds_num"], b["bin_den"], b["bin_variants"])
    if mode == MODE_COST:
        return select_cost(hist, tile_ns, b["c_fix"], b["c_byte"], b["c_reload"], b["c_flop"])
    raise ValueError("unknown table mode")
