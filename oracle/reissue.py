"""Churn recovery: re-plan failed tasks over the surviving devices (test infrastructure).

Section 4.2: a failure is a new snapshot of the scheduling problem restricted to the unfinished
shards; surviving assignments stay fixed (Section 4.1, "Solver and reuse"); the downlink term of a
candidate owner counts only the rows / columns it does not already cache and carries no latency
term; the lost work is spread over all remaining devices (Section 3.2).  The re-solve itself is,
as for the cold-start plan, a heuristic here: longest-processing-time-first list scheduling on the
cache-aware cost.
"""
from __future__ import annotations

from typing import Iterable, List, Sequence, Tuple

from .cost import ceil_div, c_comp, c_dl, c_ul, task_mem
from .plan import FLAG_REISSUED, FLAG_SUPERSEDED, Plan, PlanError, Task, split_counts


def _uncovered(lo: int, hi: int, intervals: Iterable[Tuple[int, int]]) -> int:
    """Number of integers in [lo, hi) not covered by the union of the given half-open intervals."""
    covered = 0
    cur = lo
    for a, b in sorted(intervals):
        a, b = max(a, cur), min(b, hi)
        if b > a:
            covered += b - a
            cur = b
    return (hi - lo) - covered


def reissue(plan: Plan, failed: Sequence[int]) -> List[Task]:
    """Appends the replacement tasks to `plan.tasks`, flags the failed ones superseded, records
    the dead devices per GEMM, and returns the new tasks (id order)."""
    o = plan.opts
    F = sorted(set(int(f) for f in failed))
    for f in F:
        if f < 0 or f >= len(plan.tasks):
            raise PlanError("E_RANGE", f"task id {f}")
        if plan.tasks[f].flags & FLAG_SUPERSEDED:
            raise PlanError("E_INVAL", f"task {f} already superseded")
    if not F:
        return []

    gemm_ids = sorted(set(plan.tasks[f].gemm for f in F))
    fset = set(F)
    # per GEMM: devices that died now, and the survivors (owners of live, non-failed tasks)
    survivors = {}
    for g in gemm_ids:
        dead_now = set(plan.tasks[f].dev for f in F if plan.tasks[f].gemm == g)
        dead = plan.dead[g] | dead_now
        owners = set(t.dev for t in plan.tasks
                     if t.gemm == g and not (t.flags & FLAG_SUPERSEDED) and t.id not in fset)
        live = sorted(owners - dead)
        if not live:
            raise PlanError("E_NO_DEVICES", f"GEMM {g} has no surviving device")
        survivors[g] = (live, dead)

    # pieces: each failed task cut by rows into at most R granule-aligned parts
    pieces: List[Task] = []
    next_id = len(plan.tasks)
    for f in F:
        t = plan.tasks[f]
        rows_g = ceil_div(t.alpha, o.gran_m)
        p = min(o.reissue_fanout, rows_g)
        r0 = t.m0
        for hg in split_counts(rows_g, p):
            r1 = min(t.m1, r0 + hg * o.gran_m)
            pieces.append(Task(next_id, t.gemm, -1, f, r0, r1, t.n0, t.n1, t.k0, t.k1, t.kslice,
                               FLAG_REISSUED, t.part_off + (r0 - t.m0) * t.beta, 0))
            next_id += 1
            r0 = r1

    # owners: largest piece first, to the survivor that finishes it earliest (cache-aware)
    load = {g: {k: 0 for k in survivors[g][0]} for g in gemm_ids}
    held = {g: {k: [] for k in survivors[g][0]} for g in gemm_ids}
    for t in plan.tasks:
        if t.gemm in held and t.dev in held[t.gemm] and not (t.flags & FLAG_SUPERSEDED) \
                and t.id not in fset:
            held[t.gemm][t.dev].append(t)
    for pc in sorted(pieces, key=lambda x: (-2 * x.alpha * x.beta * x.kappa, x.id)):
        best = None
        for k in survivors[pc.gemm][0]:
            d = plan.devices[k]
            if task_mem(pc.alpha, pc.beta, pc.kappa, o.b_in, o.b_out) > d.mem_bytes:
                continue
            mine = [h for h in held[pc.gemm][k] if h.k0 <= pc.k0 and h.k1 >= pc.k1]
            a_hat = _uncovered(pc.m0, pc.m1, [(h.m0, h.m1) for h in mine])
            b_hat = _uncovered(pc.n0, pc.n1, [(h.n0, h.n1) for h in mine])
            c = max(c_dl(a_hat, b_hat, pc.kappa, d, o.b_in, latency=False),
                    c_ul(pc.alpha, pc.beta, d, o.b_out),
                    c_comp(pc.alpha, pc.beta, pc.kappa, d))
            cand = load[pc.gemm][k] + c
            if best is None or cand < best[0]:
                best = (cand, k, c)
        if best is None:
            raise PlanError("E_INFEASIBLE", "no survivor can hold a reissued piece")
        _, k, c = best
        pc.dev, pc.cost_ns = k, c
        load[pc.gemm][k] += c
        held[pc.gemm][k].append(pc)

    for f in F:
        plan.tasks[f].flags |= FLAG_SUPERSEDED
    for g in gemm_ids:
        plan.dead[g] = survivors[g][1]
    plan.tasks.extend(pieces)
    return pieces


def recovery_makespan_ns(plan: Plan, new_tasks: Sequence[Task]) -> int:
    load = {}
    for t in new_tasks:
        load[(t.gemm, t.dev)] = load.get((t.gemm, t.dev), 0) + t.cost_ns
    return max(load.values()) if load else 0
