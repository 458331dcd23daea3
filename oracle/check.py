"""Independent checkers for plans and results (test infrastructure).

Coverage: Section 4.1 requires the shards to cover the whole output with no work done twice; its
sum-of-areas condition is necessary but not sufficient for a tiling, so coverage is checked directly.
Constraints: Eq. (zero-task-constraint), Eq. (memory-constraint).
Freivalds: Section 6 ("Robustness to poisoning attacks"): r^T (A B) s = (A^T r)^T (B s).
"""
from __future__ import annotations

from typing import List, Sequence

import numpy as np

from .cost import task_mem
from .plan import FLAG_SUPERSEDED, Plan


def live_tasks(plan: Plan):
    return [t for t in plan.tasks if not (t.flags & FLAG_SUPERSEDED)]


def cover_count_bruteforce(plan: Plan, gemm: int) -> np.ndarray:
    """count[i, j, k] = number of live tasks of `gemm` that contain the index triple (tiny shapes)."""
    g = plan.gemms[gemm]
    cnt = np.zeros((g.M, g.N, g.K), dtype=np.int32)
    for t in live_tasks(plan):
        if t.gemm == gemm:
            cnt[t.m0:t.m1, t.n0:t.n1, t.k0:t.k1] += 1
    return cnt


def check_cover(plan: Plan, gemm: int) -> None:
    """Exact cover at any size: K boundaries of all live tasks cut K into elementary intervals;
    inside each the live tasks' rectangles must tile M x N (area sum and pairwise disjointness
    via a painted element map of one byte per output element)."""
    g = plan.gemms[gemm]
    tasks = [t for t in live_tasks(plan) if t.gemm == gemm]
    cuts = sorted({0, g.K} | {t.k0 for t in tasks} | {t.k1 for t in tasks})
    assert cuts[0] == 0 and cuts[-1] == g.K, "K range exceeded"
    for ka, kb in zip(cuts[:-1], cuts[1:]):
        paint = np.zeros((g.M, g.N), dtype=np.uint8)
        for t in tasks:
            if t.k0 <= ka and t.k1 >= kb:
                assert 0 <= t.m0 < t.m1 <= g.M and 0 <= t.n0 < t.n1 <= g.N
                paint[t.m0:t.m1, t.n0:t.n1] += 1
            else:
                assert t.k1 <= ka or t.k0 >= kb, "task straddles a K cut"
        assert paint.min() == 1 and paint.max() == 1, \
            f"gemm {gemm} K[{ka},{kb}): cover count min {paint.min()} max {paint.max()}"


def check_constraints(plan: Plan) -> None:
    o = plan.opts
    for t in live_tasks(plan):
        assert t.alpha > 0 and t.beta > 0 and t.kappa > 0, "zero-task rule: a task has alpha, beta, kappa > 0"
        d = plan.devices[t.dev]
        assert task_mem(t.alpha, t.beta, t.kappa, o.b_in, o.b_out) <= d.mem_bytes, \
            f"task {t.id} exceeds device {t.dev} memory"


def check_arena(plan: Plan) -> None:
    """Original blocks are disjoint, 32-element aligned and inside the arena; a reissued piece is
    a row range of its parent's block."""
    spans = []
    for t in plan.tasks[:plan.n_original]:
        assert t.part_off % 32 == 0
        spans.append((t.part_off, t.part_off + t.alpha * t.beta))
    spans.sort()
    for (a0, a1), (b0, b1) in zip(spans[:-1], spans[1:]):
        assert a1 <= b0
    assert not spans or spans[-1][1] <= plan.arena_elems
    for t in plan.tasks[plan.n_original:]:
        p = plan.tasks[t.parent]
        assert (t.n0, t.n1, t.k0, t.k1) == (p.n0, p.n1, p.k0, p.k1)
        assert p.m0 <= t.m0 < t.m1 <= p.m1
        assert t.part_off == p.part_off + (t.m0 - p.m0) * p.beta


def freivalds_residual(A: np.ndarray, B: np.ndarray, C: np.ndarray, seed: int, reps: int = 4):
    """max over `reps` random +-1 vector pairs of |r^T C s - (A^T r)^T (B s)|, and the scale
    (|A^T r|)^T |B s| against which it is judged.  All fp64."""
    rng = np.random.default_rng(seed)
    worst, scale = 0.0, 0.0
    for _ in range(reps):
        r = rng.integers(0, 2, A.shape[0]).astype(np.float64) * 2 - 1
        s = rng.integers(0, 2, B.shape[1]).astype(np.float64) * 2 - 1
        lhs = r @ (C.astype(np.float64) @ s)
        u, v = A.T @ r, B @ s
        worst = max(worst, abs(lhs - u @ v))
        scale = max(scale, float(np.abs(u) @ np.abs(v)))
    return worst, scale
