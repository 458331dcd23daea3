"""Sub-GEMM execution and assembly of partial blocks on the CPU (test infrastructure).

The decomposition is exact: the union of the devices' output blocks is the output (Section 4.1,
"Search space of GEMM") and the assembled result equals the single-device GEMM (Section 3.2).
So the numerical oracle is the definition written out: every task multiplies its own rows of A and
columns of B over its own K-range in fp64; the parameter-server side then sums, for each output
element, the partial blocks of all K-slices in a fixed balanced-tree order.

Inputs are the bf16 bit patterns (uint16) of the stored operands, widened exactly to fp64.
"""
from __future__ import annotations

from typing import Dict, List, Sequence

import numpy as np

from .plan import FLAG_REISSUED, FLAG_SUPERSEDED, Plan, Task


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """bf16 is the upper half of an IEEE binary32: shift into place, reinterpret, widen."""
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def f64_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round to the nearest bf16 (8 significant bits), ties to even, in ONE rounding from fp64; the
    bit patterns as uint16.  (Going through fp32 first would round twice.)  Values are assumed to lie
    in bf16's normal range or to be zero, as every output of the workloads here does."""
    x = np.asarray(x, dtype=np.float64)
    m, e = np.frexp(x)                       # x = m * 2^e, 0.5 <= |m| < 1
    r = np.ldexp(np.rint(m * 256.0), e - 8)  # rint rounds half to even: 8 significant bits kept
    return (r.astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)


def op_a(stored: np.ndarray, transA: int) -> np.ndarray:
    """A as an [M x K] array.  transA = 1: stored is [K x M] and A[i, k] = stored[k, i]."""
    return stored.T if transA else stored


def op_b(stored: np.ndarray, transB: int) -> np.ndarray:
    """B as a [K x N] array.  transB = 1: stored is [N x K] and B[k, j] = stored[j, k]."""
    return stored.T if transB else stored


def sub_gemm(t: Task, A: np.ndarray, B: np.ndarray) -> np.ndarray:
    """P_t = A[m0:m1, k0:k1] . B[k0:k1, n0:n1] in fp64 (A is [M x K], B is [K x N])."""
    return A[t.m0:t.m1, t.k0:t.k1] @ B[t.k0:t.k1, t.n0:t.n1]


def sub_gemm_from_bits(t: Task, transA: int, transB: int, a_bits: np.ndarray, b_bits: np.ndarray) -> np.ndarray:
    """Same block as `sub_gemm`, starting from the stored bf16 bit patterns: only the task's own
    rows of A and columns of B are widened (what a device would be sent)."""
    a = a_bits[t.k0:t.k1, t.m0:t.m1].T if transA else a_bits[t.m0:t.m1, t.k0:t.k1]
    b = b_bits[t.n0:t.n1, t.k0:t.k1].T if transB else b_bits[t.k0:t.k1, t.n0:t.n1]
    return bf16_bits_to_f64(np.ascontiguousarray(a)) @ bf16_bits_to_f64(np.ascontiguousarray(b))


def execute(plan: Plan, A: Sequence[np.ndarray], B: Sequence[np.ndarray],
            task_ids=None, arena: np.ndarray = None, dropped=()) -> np.ndarray:
    """Runs tasks (all live ones by default) and writes each block, row-major with leading
    dimension beta, at its offset in the packed arena (fp64).  Unwritten cells stay NaN."""
    if arena is None:
        arena = np.full(plan.arena_elems, np.nan, dtype=np.float64)
    dropped = set(int(x) for x in dropped)
    ids = range(len(plan.tasks)) if task_ids is None else task_ids
    for i in ids:
        t = plan.tasks[i]
        if (t.flags & FLAG_SUPERSEDED) or i in dropped:
            continue
        P = sub_gemm(t, A[t.gemm], B[t.gemm])
        arena[t.part_off:t.part_off + t.alpha * t.beta] = P.reshape(-1)
    return arena


def tree_sum(parts: List[np.ndarray]) -> np.ndarray:
    """Balanced pairwise sum of adjacent slices; the list is padded to a power of two with +0.0
    (the order a butterfly exchange over slice index gives).  dtype follows the inputs."""
    n = 1
    while n < len(parts):
        n *= 2
    zero = np.zeros_like(parts[0])
    level = list(parts) + [zero] * (n - len(parts))
    while len(level) > 1:
        level = [level[i] + level[i + 1] for i in range(0, len(level), 2)]
    return level[0]


def assemble(plan: Plan, arena: np.ndarray, dtype=np.float64) -> List[np.ndarray]:
    """C_g[i, j] = tree-sum over the K-slices s of the partial block that covers (i, j) in slice s.

    Only original tasks are read: a reissued piece writes into its parent's block, so the arena
    layout never changes.  `dtype=np.float32` emulates the GPU's fp32 adds bit for bit."""
    return [assemble_gemm(plan, arena, gi, dtype) for gi in range(len(plan.gemms))]


def assemble_gemm(plan: Plan, arena: np.ndarray, gi: int, dtype=np.float64) -> np.ndarray:
    """`assemble` for one GEMM of the plan."""
    arena = arena.astype(dtype, copy=False)
    g = plan.gemms[gi]
    S = plan.ksplit[gi]
    slabs = [np.full((g.M, g.N), np.nan, dtype=dtype) for _ in range(S)]
    for t in plan.tasks[:plan.n_original]:
        if t.gemm != gi:
            continue
        blk = arena[t.part_off:t.part_off + t.alpha * t.beta].reshape(t.alpha, t.beta)
        slabs[t.kslice][t.m0:t.m1, t.n0:t.n1] = blk
    return tree_sum(slabs)


def gemm_direct(A: np.ndarray, B: np.ndarray) -> np.ndarray:
    """The undecomposed GEMM in fp64."""
    return A @ B


def abs_bound(A: np.ndarray, B: np.ndarray) -> np.ndarray:
    """(|A| |B|)_ij, the scale of the elementwise acceptance bound."""
    return np.abs(A) @ np.abs(B)


def sample_entries(A: np.ndarray, B: np.ndarray, rows: np.ndarray, cols: np.ndarray):
    """C[i, j] and (|A||B|)[i, j] for the listed (i, j) pairs, one fp64 dot product each."""
    a = A[rows, :]
    b = B[:, cols].T
    return np.einsum("ik,ik->i", a, b), np.einsum("ik,ik->i", np.abs(a), np.abs(b))
