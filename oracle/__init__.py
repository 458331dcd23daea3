"""CPU oracle for the Cleave hot path -- TEST INFRASTRUCTURE, not a product path.

Plain, slow, obviously-correct Python/NumPy code written from the paper: the planner (integer
only), the churn re-planner, the per-task fp64 sub-GEMMs, the assembly of K-split partial blocks,
and independent checkers.  It shares no code with the CUDA library and never imports it; only
tests, the smoke check and the benchmark's `cpu_baseline` / `--impl reference` legs may import it.

Parity status of each part (what pins it besides itself):
  cost.py      pinned  - the per-level costs and the 16.6 s per-batch figure of the paper's worked
                         example (Section 5.2), reproduced from the cost equations of Section 4.1
  plan.py      pinned for feasibility (exact cover by brute force, memory and zero-task
                         constraints, homogeneous devices -> equal grid, makespan >= Eq. 18 bound);
               "parity unpinned" for optimality: the paper's solver (a commercial MILP solver)
                         is not specified as an algorithm, so the quality of the heuristic plan
                         against the paper's optimum cannot be pinned
  reissue.py   pinned for semantics (survivors fixed, dead devices excluded, failed rectangles
                         covered exactly once, cache-aware downlink reduces to zero for cached
                         rows/columns); optimality "parity unpinned" as above
  numerics.py  pinned  - assembled result == undecomposed GEMM (brute force, triple loop, on
                         tiny shapes; bit-exact on small-integer inputs; numpy float64 matmul)
"""
