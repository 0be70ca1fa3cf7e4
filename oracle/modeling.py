"""Routing-skew modelling: Effective Experts of a probability vector, the binary
search for the Dirichlet concentration (Algorithm 1), the ddist:X notation and
the exemplar of a routing distribution.

TEST INFRASTRUCTURE ONLY.  Nothing on the product path may import this module;
it shares no code with the CUDA library.

What the paper fixes
  * eff_exp = (sum t)^2 / sum t^2                               (Section III-A, Eq. 2)
  * Algorithm 1: bisection on alpha over [1e-6, 1e6] with the arithmetic
    midpoint; at each step draw S vectors from Dir(alpha_mid), average their
    eff_exp, move lo up when the average is below the target and hi down
    otherwise; the result is the last midpoint                   (Algorithm 1)
  * ddist:X names Dir(alpha) whose target is eff_exp* = E / X    (Section III-A)
  * an exemplar is the per-expert token-count vector sorted in descending order
    and scaled to unit L2 norm; with several samples the centroid is used
                                                                  (Section IV-A)
Readings taken where the paper is silent
  * Algorithm 1 applies eff_exp to the sampled probability vectors, as printed;
  * the Dirichlet draws come from a caller-supplied sampler, so the search can
    run on common random numbers and be deterministic;
  * the centroid of unit vectors is rescaled to unit length, then stored as
    round(e_i * 2^30).
"""
from __future__ import annotations

import numpy as np


def eff_exp(t) -> float:
    """Eq. 2 on any non-negative vector (counts or probabilities), in fp64."""
    t = np.asarray(t, dtype=np.float64)
    s2 = float(np.sum(t * t))
    if s2 == 0.0:
        return 0.0
    s1 = float(np.sum(t))
    return s1 * s1 / s2


def ddist_target(E: int, X: float) -> float:
    """Target Effective Experts of ddist:X."""
    return E / X


def binary_search_alpha(target: float, E: int, S: int, iters: int, draw,
                        alpha_min: float = 1e-6, alpha_max: float = 1e6) -> float:
    """Algorithm 1.  ``draw(alpha, E, S)`` returns S probability vectors [S, E]."""
    lo, hi = alpha_min, alpha_max
    mid = (lo + hi) / 2.0
    for _ in range(iters):
        mid = (lo + hi) / 2.0
        p = draw(mid, E, S)
        v = sum(eff_exp(p[s]) for s in range(S)) / S
        if v < target:
            lo = mid          # too skewed: raise alpha
        else:
            hi = mid          # too uniform: lower alpha
    return mid


def sorted_unit_vector(counts) -> np.ndarray:
    """Descending sort, then division by the L2 norm."""
    q = np.sort(np.asarray(counts, dtype=np.float64))[::-1]
    n = float(np.sqrt(np.sum(q * q)))
    return q / n if n > 0 else q


def exemplar(count_vectors) -> np.ndarray:
    """Centroid of the samples' sorted unit vectors, rescaled to unit norm."""
    vs = [sorted_unit_vector(c) for c in count_vectors]
    c = np.zeros_like(vs[0])
    for v in vs:
        c = c + v
    c = c / len(vs)
    n = float(np.sqrt(np.sum(c * c)))
    return c / n if n > 0 else c


def exemplar_q30(count_vectors) -> np.ndarray:
    """The exemplar in the fixed-point form the dispatcher scores with."""
    return np.rint(exemplar(count_vectors) * float(1 << 30)).astype(np.int64)


def cosine(a, b) -> float:
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    return float(np.dot(a, b) / (np.sqrt(np.dot(a, a)) * np.sqrt(np.dot(b, b))))
