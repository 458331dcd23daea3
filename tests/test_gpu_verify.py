"""Block verification on the GPU (cleave_verify) against the oracle, and its behaviour on honest,
corrupted and missing blocks."""
import numpy as np
import pytest

import cleave_inputs as ci
from helpers import GpuRun, lib_plan_for, oracle_operands, oracle_plan_for
from oracle import numerics as nm, verify as ov

pytestmark = pytest.mark.gpu


def test_values_match_oracle_on_oracle_made_blocks():
    """The arena is filled with the ORACLE's blocks (rounded to fp32), so both sides check the same
    data; lhs, rhs and scale of every task must agree to fp32 summation accuracy, in all layouts."""
    import torch
    w = ci.config(2, 8)                                 # fwd, dgrad, wgrad GEMMs, several K-slices
    ts = ci.make_tensors(w)
    p, op = lib_plan_for(w), oracle_plan_for(w)
    A, B = oracle_operands(w, ts)
    arena64 = nm.execute(op, A, B)
    arena32 = np.nan_to_num(arena64).astype(np.float32)  # padding between blocks is never read
    run = GpuRun(w, ts, p)
    run.partials.copy_(torch.from_numpy(arena32))
    bad, vals = p.verify(run.A, run.B, run.partials, seed=1234)
    assert bad == 0 and vals.shape == (p.num_tasks, 4)
    for t in op.tasks:
        P = arena32[t.part_off:t.part_off + t.alpha * t.beta].reshape(t.alpha, t.beta)
        lhs, rhs, scale = ov.task_check(t, A[t.gemm], B[t.gemm], P, seed=1234)
        tol = 2e-6 * scale + 1e-6
        assert abs(vals[t.id, 0] - lhs) <= tol and abs(vals[t.id, 1] - rhs) <= tol, t.id
        assert abs(vals[t.id, 2] - scale) <= 1e-4 * scale and vals[t.id, 3] == 0.0


def test_honest_blocks_pass_and_corruption_is_caught():
    import torch
    w = ci.config(4, 8)
    ts = ci.make_tensors(w)
    p = lib_plan_for(w)
    run = GpuRun(w, ts, p)
    run.exec()
    bad, vals = p.verify(run.A, run.B, run.partials, seed=7)
    assert bad == 0
    assert np.all(np.abs(vals[:, 0] - vals[:, 1]) <= 2e-6 * vals[:, 2] + 1e-6)     # far inside the threshold

    tasks = p.tasks()
    victim = int(tasks["id"][len(tasks) // 3])
    off = int(tasks["part_off"][victim]) + 5
    run.partials[off] += 0.5                            # one changed entry of one returned block
    bad, vals = p.verify(run.A, run.B, run.partials, seed=7)
    assert bad == 1 and vals[victim, 3] == 1.0 and vals[:, 3].sum() == 1.0
    assert abs(abs(vals[victim, 0] - vals[victim, 1]) - 0.5) < 1e-2                  # +-1 vectors: residual = the change
    run.partials[off] -= 0.5

    failed = ci.make_failed_ids(p.num_tasks, w.fail_frac, w.seed + 2)
    p.set_drops(failed)
    run.partials.fill_(float("nan"))
    run.exec()                                          # dropped tasks leave their blocks unwritten
    bad, vals = p.verify(run.A, run.B, run.partials, seed=8)
    assert bad == len(failed) and set(np.nonzero(vals[:, 3])[0].tolist()) == set(failed.tolist())
    run.reissue(failed)
    bad, vals = p.verify(run.A, run.B, run.partials, seed=9)
    assert bad == 0 and vals.shape[0] == p.num_tasks    # replacement pieces are checked, superseded tasks skipped
    assert np.all(vals[failed, 2] == 0.0)


def test_fused_mode_reads_one_slice_blocks_from_c():
    w = ci.config(3, 8)
    ts = ci.make_tensors(w)
    p = lib_plan_for(w)
    run = GpuRun(w, ts, p)
    run.exec_fused()
    bad, _ = p.verify(run.A, run.B, run.partials, seed=3)
    assert bad == 0
    gi = [i for i in range(p.n_gemms) if p.ksplit(i) == 1][0]
    run.C[gi][17, 33] += 1.0                            # corrupt a directly written block
    bad, vals = p.verify(run.A, run.B, run.partials, seed=3)
    t = p.tasks()
    hit = [int(x["id"]) for x in t if x["gemm"] == gi and x["m0"] <= 17 < x["m1"] and x["n0"] <= 33 < x["n1"]]
    assert bad == 1 and vals[hit[0], 3] == 1.0
