"""Shared test helpers: bit views of torch tensors, seeded cases, comparisons."""
from __future__ import annotations

import numpy as np
import torch

import damoe_inputs as di


def bits16(t: torch.Tensor) -> np.ndarray:
    """bf16 torch tensor (any device) -> uint16 numpy bit patterns."""
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def from_bits16(b: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(b).view(np.int16)).view(torch.bfloat16)


class Case:
    """One seeded synthetic batch: routing + activations + (lazy) weights."""

    def __init__(self, seed, T, E, k, H, I, alpha):
        self.seed, self.T, self.E, self.k, self.H, self.I, self.alpha = seed, T, E, k, H, I, alpha
        self.ids, self.w, self.p = di.routing_batch(seed, T, k, E, alpha)
        self.weights = di.MoEWeights(seed if E <= 8 else 12345, E, H, I)

    def x(self, device="cpu"):
        return di.activations(self.seed, self.T, self.H, device)

    def w13_bits(self, e):
        return bits16(self.weights.expert_w13(e))

    def w2_bits(self, e):
        return bits16(self.weights.expert_w2(e))


def config0(seed=0, T=64):
    return Case(seed, T, 8, 2, 1024, 512, 1.0)


def rel_frobenius(a: np.ndarray, ref: np.ndarray) -> float:
    a = np.asarray(a, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    return float(np.linalg.norm(a - ref) / max(np.linalg.norm(ref), 1e-300))


def max_scaled_err(a: np.ndarray, ref: np.ndarray) -> float:
    """max |a - ref| / max(1, |ref|)."""
    a = np.asarray(a, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    return float(np.max(np.abs(a - ref) / np.maximum(1.0, np.abs(ref))))
