"""Full-size parity in the launch configuration the benchmark times (Llama-7B-shaped layer,
1024 devices): outputs the oracle can compute one by one, plus a Freivalds identity over the whole
of every C."""
import numpy as np
import pytest

import cleave_inputs as ci
from helpers import GpuRun, lib_plan_for
from oracle import check, numerics as nm

pytestmark = pytest.mark.gpu


def _check_against_oracle(w, ts, run, freivalds_reps=2):
    rng = np.random.default_rng(7)
    wide = {}
    for gi, g in enumerate(w.gemms):
        for key in (g.a_key, g.b_key):
            if key not in wide:
                wide[key] = nm.bf16_bits_to_f64(ci.bf16_bits(ts[key]))
        A, B = nm.op_a(wide[g.a_key], g.transA), nm.op_b(wide[g.b_key], g.transB)
        C = run.C[gi].cpu().numpy()
        # 512 sampled entries, among them the four corners and tile-edge neighbours
        rows = np.concatenate([rng.integers(0, g.M, 500), [0, 0, g.M - 1, g.M - 1, 127, 128, 255, 256, 127, 128, 129, 63]])
        cols = np.concatenate([rng.integers(0, g.N, 500), [0, g.N - 1, 0, g.N - 1, 255, 256, 127, 128, 128, 127, 1, 64]])
        ref, bound = nm.sample_entries(A, B, rows, cols)
        got = C[rows, cols].astype(np.float64)
        assert np.all(np.abs(got - ref) <= 1e-2 * bound), g.name
        assert np.linalg.norm(got - ref) <= 1e-3 * np.linalg.norm(ref), g.name
        worst, scale = check.freivalds_residual(A, B, C, seed=gi, reps=freivalds_reps)
        assert worst <= 1e-3 * scale, g.name     # any lost or doubled block shifts r^T C s far beyond rounding


def test_config3_sampled_entries_and_freivalds():
    """Llama-7B-shaped layer, 1024 devices, the launch configuration the benchmark times (fused
    write-out of one-slice GEMMs)."""
    import torch
    w = ci.config(3)
    ts = ci.make_tensors(w)
    p = lib_plan_for(w)
    run = GpuRun(w, ts, p)
    run.exec_fused(); run.assemble(); p.check_status()
    torch.cuda.synchronize()
    _check_against_oracle(w, ts, run)
    bad, vals = p.verify(run.A, run.B, run.partials, seed=5)     # every returned block passes the vector check
    assert bad == 0 and np.all(np.abs(vals[:, 0] - vals[:, 1]) <= 5e-6 * vals[:, 2] + 1e-5)
    # the mode the benchmark times (blocks that complete a cell are used up on arrival): the same bits
    keep = [c.clone() for c in run.C]
    for c in run.C:
        c.fill_(float("nan"))
    run.exec_opts(direct=True, finish=True, consume=True); run.assemble(); p.check_status()
    torch.cuda.synchronize()
    for g, a, b in zip(w.gemms, keep, run.C):
        assert torch.equal(a.view(torch.int32), b.view(torch.int32)), g.name


def test_config4_churn_full_size():
    """Same layer with 10 % of the tasks failed mid-step: the re-planned, reissued and re-assembled
    result equals the no-failure result bit for bit and matches the oracle; the task list after the
    re-plan equals the oracle's."""
    import torch
    from helpers import oracle_plan_for, task_matrix_lib, task_matrix_oracle
    from oracle.reissue import reissue as oracle_reissue
    w = ci.config(4)
    ts = ci.make_tensors(w)
    p = lib_plan_for(w)
    run = GpuRun(w, ts, p)
    run.exec(); run.assemble(); p.check_status()
    torch.cuda.synchronize()
    good = [c.clone() for c in run.C]
    failed = ci.make_failed_ids(p.num_tasks, w.fail_frac, w.seed + 2)
    p.set_drops(failed)
    run.partials.fill_(float("nan"))
    for c in run.C:
        c.fill_(float("nan"))
    run.exec(); run.assemble()
    assert p.status() == -9
    run.reissue(None)                                  # the bookkeeping finds the unfinished tasks itself
    run.assemble()
    assert p.status() == 0
    torch.cuda.synchronize()
    for g, a, b in zip(w.gemms, good, run.C):
        assert torch.equal(a.view(torch.int32), b.view(torch.int32)), g.name
    op = oracle_plan_for(w)
    oracle_reissue(op, failed)
    assert np.array_equal(task_matrix_lib(p), task_matrix_oracle(op))
    _check_against_oracle(w, ts, run, freivalds_reps=1)


def test_config5_sampled_entries():
    """Llama-13B-shaped layer, 4096 devices: many small tasks, up to four K-slices."""
    import torch
    w = ci.config(5)
    ts = ci.make_tensors(w)
    p = lib_plan_for(w)
    assert p.num_tasks > 30000 and max(p.ksplit(i) for i in range(p.n_gemms)) >= 4
    run = GpuRun(w, ts, p)
    run.exec_fused(); run.assemble(); p.check_status()
    torch.cuda.synchronize()
    done = p.done_counts()
    assert (done == np.array([p.task_num_tiles(i) for i in range(p.num_tasks)])).all()
    _check_against_oracle(w, ts, run, freivalds_reps=1)


def test_config2_every_output_against_the_full_oracle():
    """GPT-2-small-shaped layer at full size (12 GEMMs, 64 devices, 0.35 TFLOP): small enough for the
    oracle to compute every block, so every output element is compared, not a sample."""
    from helpers import assert_within_tolerance, oracle_operands, oracle_plan_for, task_matrix_lib, task_matrix_oracle
    w = ci.config(2)
    ts = ci.make_tensors(w)
    p, op = lib_plan_for(w), oracle_plan_for(w)
    assert np.array_equal(task_matrix_lib(p), task_matrix_oracle(op))
    A, B = oracle_operands(w, ts)
    ref = nm.assemble(op, nm.execute(op, A, B))
    run = GpuRun(w, ts, p)
    run.exec_fused(); run.assemble(); p.check_status()
    for g, got, want, a, b in zip(w.gemms, run.results(), ref, A, B):
        assert_within_tolerance(got, want, nm.abs_bound(a, b), what=g.name)
