"""Verification of returned blocks on the CPU (test infrastructure; see oracle/__init__.py).

Section 6, "Robustness to poisoning attacks": the server dispatched A' and B' and received the
block P, so it can test P = A' B' with two random vectors and three matrix-vector products instead
of a GEMM.  The paper prints the identity as r^T (A B) s = (A r)^T (B s); with A' of shape
alpha x kappa the product A' r is not defined for r of length alpha, so it is read as
r^T P s = (A'^T r)^T (B' s).

The vectors have entries +-1 drawn from a counter-based generator so that both implementations
draw the same ones: entry e of vector v (0 = r, 1 = s) of task t is the top bit of
SplitMix64's output function applied to seed + (t << 33 | e << 1 | v)  (Steele, Lea, Flood, "Fast
splittable pseudorandom number generators", OOPSLA 2014).
"""
from __future__ import annotations

import numpy as np

MASK = (1 << 64) - 1


def splitmix64_mix(x: int) -> int:
    """Output of a SplitMix64 generator whose state was x before the call."""
    z = (x + 0x9E3779B97F4A7C15) & MASK
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & MASK
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & MASK
    return z ^ (z >> 31)


def signs(seed: int, task: int, which: int, n: int) -> np.ndarray:
    """n entries of +-1.0 (fp64)."""
    out = np.empty(n, dtype=np.float64)
    for e in range(n):
        out[e] = -1.0 if splitmix64_mix((seed + ((task << 33) | (e << 1) | which)) & MASK) >> 63 else 1.0
    return out


def task_check(t, A: np.ndarray, B: np.ndarray, P: np.ndarray, seed: int):
    """(lhs, rhs, scale) for task t: lhs = r^T P s, rhs = (A'^T r) . (B' s), scale = |A'^T r| . |B' s|.
    A is [M x K], B is [K x N] (fp64), P the task's alpha x beta block as returned."""
    r, s = signs(seed, t.id, 0, t.alpha), signs(seed, t.id, 1, t.beta)
    u = A[t.m0:t.m1, t.k0:t.k1].T @ r
    v = B[t.k0:t.k1, t.n0:t.n1] @ s
    return float(r @ (P.astype(np.float64) @ s)), float(u @ v), float(np.abs(u) @ np.abs(v))
