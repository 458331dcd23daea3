"""Level-order execution of a DAG of GEMMs and its level-wise cost (test infrastructure; see
oracle/__init__.py).

Section 4.1, "Problem definition and objective": the GEMMs of a training step are processed in
level order; the GEMMs of a level are independent and run in parallel, the outputs of a level are
the inputs of the next, so a level starts when the one before it has finished.  The cost of GEMM p
of level s is that of its slowest device, C(s, p) = max_k C(s, p, k); the cost of the step up to
level s is C(0) = max_p C(0, p), C(s) = C(s - 1) + max_p C(s, p)  (equation "level-cost-s").
"""
from __future__ import annotations

from typing import Dict, List, Sequence

import numpy as np

from . import numerics as nm
from .plan import Plan


def level_costs(gemm_cost_ns: Sequence[int], levels: Sequence[int]) -> List[int]:
    """C(s) for s = 0 .. max level, from the cost C(s, p) of every GEMM and its level.  A level
    without GEMMs adds nothing."""
    n_levels = max(levels) + 1 if len(levels) else 0
    worst = [0] * n_levels
    for c, s in zip(gemm_cost_ns, levels):
        worst[s] = max(worst[s], c)
    out, total = [], 0
    for s in range(n_levels):
        total += worst[s]
        out.append(total)
    return out


def plan_level_costs(plan: Plan, levels: Sequence[int]) -> List[int]:
    """C(s) of a plan: C(s, p) is the plan's modelled makespan of GEMM p (the largest device load)."""
    return level_costs(plan.makespan_ns, levels)


def execute_levels(plan: Plan, specs, tensor_bits: Dict[str, np.ndarray], out_bf16: bool = True):
    """Runs the GEMMs level by level.  `specs[g]` names the stored operands of GEMM g (`a_key`,
    `b_key`, `transA`, `transB`), its `level`, and `out_key`, the name under which its result, rounded
    to bf16, becomes an operand of higher levels (None: a final output).  `tensor_bits`: bf16 bit
    patterns of the step's inputs.  Returns (C per GEMM in fp64 -- the value before any rounding --,
    bit patterns of every produced tensor)."""
    bits = dict(tensor_bits)
    arena = np.full(plan.arena_elems, np.nan, dtype=np.float64)
    n = len(specs)
    C: List[np.ndarray] = [None] * n
    for level in sorted({s.level for s in specs}):
        members = [g for g in range(n) if specs[g].level == level]
        A: List[np.ndarray] = [None] * n
        B: List[np.ndarray] = [None] * n
        for g in members:
            A[g] = nm.op_a(nm.bf16_bits_to_f64(bits[specs[g].a_key]), specs[g].transA)
            B[g] = nm.op_b(nm.bf16_bits_to_f64(bits[specs[g].b_key]), specs[g].transB)
        ids = [t.id for t in plan.tasks if t.gemm in set(members)]
        nm.execute(plan, A, B, task_ids=ids, arena=arena)
        for g in members:                      # the level is complete: its outputs become inputs
            C[g] = nm.assemble_gemm(plan, arena, g)
            if specs[g].out_key is not None:
                assert specs[g].out_key not in bits, "a tensor is produced once"
                bits[specs[g].out_key] = nm.f64_to_bf16_bits(C[g]) if out_bf16 else None
    return C, bits
