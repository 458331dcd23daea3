"""The exec kernel's own write-out paths against the two-step path and the oracle: the in-kernel
sum of K-split cells, bf16 outputs, DAG levels inside one launch, the orderly give-up of a wait
that runs out, and blocks of odd numbers of 128-row granules sharing CTA pairs.  Needs a B200."""
import numpy as np
import pytest

import cleave_inputs as ci
from helpers import (GpuRun, assert_within_tolerance, lib_plan_for, oracle_operands, oracle_plan_for,
                     task_matrix_lib, task_matrix_oracle)
from oracle import numerics as nm
from oracle.levels import execute_levels, plan_level_costs

pytestmark = pytest.mark.gpu


def _two_step(w, ts, **opts):
    p = lib_plan_for(w, **opts)
    run = GpuRun(w, ts, p)
    run.exec(); run.assemble(); p.check_status()
    return run.results()


@pytest.mark.parametrize("opts", [dict(kslice_max=512), dict(kslice_max=256), dict(kslice_max=512, gran_m=256), dict(ksplit=8, kslice_max=0)])
def test_in_kernel_sum_of_k_split_cells_is_bit_identical(opts):
    """Every GEMM finished by the exec kernel itself (one-slice blocks stored in C, K-split cells
    summed by the block that arrives last): no assembly kernel runs, and the bits equal those of
    cleave_exec + cleave_assemble whichever block came last."""
    w = ci.config(4, 8)
    ts = ci.make_tensors(w)
    good = _two_step(w, ts, **opts)
    p = lib_plan_for(w, **opts)
    S = [p.ksplit(i) for i in range(p.n_gemms)]
    assert max(S) >= 2
    run = GpuRun(w, ts, p)                             # C and arena start as NaN
    for rep in range(3):                               # arrival order differs from run to run
        for c in run.C:
            c.fill_(float("nan"))
        run.exec_fused(); run.assemble(); p.check_status()
        assert p.num_launches == 5                     # clear, arm, exec, clear verdict, bookkeeping check
        for g, a, b in zip(w.gemms, good, run.results()):
            assert np.array_equal(a.view(np.uint32), b.view(np.uint32)), (rep, g.name)
    done = p.done_counts()
    assert all(done[i] == p.task_num_tiles(i) for i in range(p.num_tasks))


def test_blocks_used_up_on_arrival():
    """CLEAVE_EXEC_CONSUME: the block that completes a cell is added to the others on its way out and
    never stored -- same bits in C, one block per cell missing from the arena; with a task dropped the
    flag is ignored and the usual recovery works."""
    import paper_2512_22142_b200 as cl
    w = ci.config(4, 8)
    ts = ci.make_tensors(w)
    opts = dict(kslice_max=512)
    good = _two_step(w, ts, **opts)
    p = lib_plan_for(w, **opts)
    run = GpuRun(w, ts, p)
    run.exec_opts(direct=True, finish=True, consume=True); run.assemble(); p.check_status()
    assert p.num_launches == 5
    for g, a, b in zip(w.gemms, good, run.results()):
        assert np.array_equal(a.view(np.uint32), b.view(np.uint32)), g.name
    # the arena started as NaN: in every cell of a K-split GEMM at most one slice's block is missing (the one
    # that completed the cell; which strips find their cell complete on arrival depends on timing)
    t = p.tasks()
    arena = run.partials.cpu().numpy()
    for gi, g in enumerate(w.gemms):
        if p.ksplit(gi) == 1:
            continue
        missing = np.zeros((g.M, g.N), dtype=np.int32)
        for x in t[t["gemm"] == gi]:
            a_, b_ = int(x["m1"] - x["m0"]), int(x["n1"] - x["n0"])
            blk = arena[int(x["part_off"]):int(x["part_off"]) + a_ * b_].reshape(a_, b_)
            missing[int(x["m0"]):int(x["m1"]), int(x["n0"]):int(x["n1"])] += np.isnan(blk)
        assert missing.max() <= 1, g.name
    with pytest.raises(cl.CleaveError) as e:
        p.verify(run.A, run.B, run.partials, seed=1)
    assert e.value.code == -2
    with pytest.raises(cl.CleaveError) as e:
        run.reissue([0])
    assert e.value.code == -1
    # a dropped task: every block that runs is stored, the assembly kernel sums after the reissue
    failed = ci.make_failed_ids(p.num_tasks, w.fail_frac, w.seed + 2)
    p.set_drops(failed)
    run.partials.fill_(float("nan"))
    for c in run.C:
        c.fill_(float("nan"))
    run.exec_opts(direct=True, finish=True, consume=True); run.assemble()
    assert p.status() == -9
    run.reissue(failed); run.assemble()
    assert p.status() == 0
    for g, a, b in zip(w.gemms, good, run.results()):
        assert np.array_equal(a.view(np.uint32), b.view(np.uint32)), g.name


def test_unequal_slices_fall_back_to_the_assembly_kernel():
    """Blocks off the 128-grid (granule 64) under memory budgets so small that the K-slices of a block
    are repaired into different pieces: such a GEMM cannot be summed cell by cell in the exec kernel
    and goes through cleave_assemble; the result is the same.  (On the 128-grid the kernel's cells do
    not depend on the blocks' shapes: the same budgets with granule 128 need no assembly kernel.)"""
    gemms, tensors = ci.projection_gemms(512, [("p", 512, 384)], ("fwd", "wgrad"))
    w = ci.Workload("tight", gemms, tensors, n_devices=12, mem_range=(150_000, 3_000_000), seed=0)
    ts = ci.make_tensors(w, integer=True)
    on_grid = lib_plan_for(w, kslice_max=128, gran_m=128, gran_n=128, gran_k=64)
    assert on_grid.finishable(0) and on_grid.finishable(1)
    opts = dict(kslice_max=128, gran_m=64, gran_n=64, gran_k=64)
    p, op = lib_plan_for(w, **opts), oracle_plan_for(w, **opts)
    assert np.array_equal(task_matrix_lib(p), task_matrix_oracle(op))
    assert p.ksplit(0) == 4 and not p.finishable(0) and not p.finishable(1)
    A, B = oracle_operands(w, ts)
    ref = nm.assemble(op, nm.execute(op, A, B))
    run = GpuRun(w, ts, p)
    run.exec_fused(); run.assemble(); p.check_status()
    assert p.num_launches > 5                          # the assembly kernel did run
    for g, got, want in zip(w.gemms, run.results(), ref):
        assert np.array_equal(got.astype(np.float64), want), g.name


def _bf16_close(got_bits, ref64, bound, what):
    """bf16 outputs against the oracle's fp64 result: the kernel rounds its fp32 sum once, so an
    output lies within half a bf16 unit in the last place (2^-9 relative) of a value that itself is
    within the fp32 accumulation error (a few 2^-24 of (|A||B|)_ij) of the exact sum; almost all
    outputs equal the exact sum rounded once."""
    got = nm.bf16_bits_to_f64(got_bits)
    assert np.isfinite(got).all(), what
    err = np.abs(got - ref64)
    assert (err <= 2.0 ** -8 * np.abs(ref64) + 1e-5 * bound).all(), f"{what}: {err.max():.3e}"
    same = got_bits == nm.f64_to_bf16_bits(ref64)
    assert same.mean() > 0.99, f"{what}: {1 - same.mean():.4f} of the outputs differ from the rounded exact sum"


def test_bf16_outputs_match_the_rounded_oracle():
    w = ci.config(2, 4)
    ts = ci.make_tensors(w)
    p, op = lib_plan_for(w, kslice_max=512), oracle_plan_for(w, kslice_max=512)
    A, B = oracle_operands(w, ts)
    ref = nm.assemble(op, nm.execute(op, A, B))
    run = GpuRun(w, ts, p, bf16_out=True)
    run.exec_opts(direct=True, finish=True, bf16=True); run.assemble(); p.check_status()
    fused = run.results()
    for gi, (g, got, want) in enumerate(zip(w.gemms, fused, ref)):
        _bf16_close(got, want, nm.abs_bound(A[gi], B[gi]), g.name)
    # the two-step path with bf16 outputs rounds the same fp32 sums: identical bits
    run2 = GpuRun(w, ts, lib_plan_for(w, kslice_max=512), bf16_out=True)
    run2.exec_opts(bf16=True); run2.assemble(); run2.plan.check_status()
    for g, a, b in zip(w.gemms, fused, run2.results()):
        assert np.array_equal(a, b), g.name
    # integer inputs: every sum is exact, so the rounded outputs are equal bit for bit
    ts = ci.make_tensors(w, integer=True)
    A, B = oracle_operands(w, ts)
    ref = nm.assemble(op, nm.execute(op, A, B))
    run3 = GpuRun(w, ts, lib_plan_for(w, kslice_max=512), bf16_out=True)
    run3.exec_opts(direct=True, finish=True, bf16=True); run3.assemble(); run3.plan.check_status()
    for g, got, want in zip(w.gemms, run3.results(), ref):
        assert np.array_equal(got, nm.f64_to_bf16_bits(want)), g.name


def _chain(tokens=640, d0=256, d1=384, d2=256, n_devices=6):
    gemms, tensors, produced = ci.two_branch_chain(tokens, d0, d1, d2)
    return ci.Workload("chain", gemms, tensors, n_devices=n_devices, mem_range=(64 * ci.MB, ci.GB), produced=produced)


@pytest.mark.parametrize("integer", [True, False])
def test_dag_levels_inside_one_launch(integer):
    """Three levels in one launch: level-1 and level-2 GEMMs read, as A and B operands in both
    layouts, the bf16 outputs that level-0 GEMMs wrote moments before (the contraction of the level-2
    GEMM is K-split and summed in the kernel)."""
    w = _chain()
    ts = ci.make_tensors(w, integer=integer)
    opts = dict(kslice_max=256)
    p, op = lib_plan_for(w, **opts), oracle_plan_for(w, **opts)
    assert np.array_equal(task_matrix_lib(p), task_matrix_oracle(op))
    assert p.num_levels == 3 and max(p.ksplit(i) for i in range(p.n_gemms)) >= 2
    levels = [g.level for g in w.gemms]
    want_cost = plan_level_costs(op, levels)
    assert [p.level_makespan_ns(s) for s in range(3)] == [want_cost[0], want_cost[1] - want_cost[0], want_cost[2] - want_cost[1]]
    assert p.step_makespan_ns == want_cost[-1]
    ref, ref_bits = execute_levels(op, w.gemms, {k: ci.bf16_bits(t) for k, t in ts.items()})
    run = GpuRun(w, ts, p, bf16_out=True)
    for rep in range(2):
        for c in run.C:
            c.fill_(float("nan"))
        run.exec_opts(direct=True, finish=True, bf16=True); run.assemble(); p.check_status()
        out = run.results()
        for gi, g in enumerate(w.gemms):
            if integer:
                assert np.array_equal(out[gi], nm.f64_to_bf16_bits(ref[gi])), (rep, g.name)
            else:
                got = nm.bf16_bits_to_f64(out[gi])
                d = got - ref[gi]
                # bf16 storage of the result (2^-9 relative) on top of the path's own tolerance
                assert np.linalg.norm(d) <= 4e-3 * np.linalg.norm(ref[gi]), g.name
    # only the higher levels again (what follows the recovery of a level): same outputs
    keep = [c.clone() for c in run.C]
    for g, c in zip(w.gemms, run.C):
        if g.level >= 1:
            c.fill_(float("nan"))
    run.exec_opts(direct=True, finish=True, bf16=True, level_begin=1); p.check_status()
    import torch
    torch.cuda.synchronize()
    for g, a, b in zip(w.gemms, keep, run.C):
        assert torch.equal(a.view(torch.int16), b.view(torch.int16)), g.name


def test_a_wait_that_runs_out_ends_the_kernel_in_order():
    """With a wait limit of zero the first wait that is not satisfied at once gives up: the kernel
    returns, the status says E_TIMEOUT, tasks show as unfinished, and the next ordinary execution on
    the same plan is exact.  Nothing here faults or hangs: every role leaves its loop and both CTAs
    of each pair meet at the final barrier."""
    w = ci.config(2, 8)
    ts = ci.make_tensors(w, integer=True)
    p, op = lib_plan_for(w), oracle_plan_for(w)
    A, B = oracle_operands(w, ts)
    ref = nm.assemble(op, nm.execute(op, A, B))
    run = GpuRun(w, ts, p)
    p.set_wait_limit_ns(0)
    run.exec()
    assert p.status() == -7                                # E_TIMEOUT
    done = p.done_counts()
    assert (done < np.array([p.task_num_tiles(i) for i in range(p.num_tasks)])).any()
    p.set_wait_limit_ns(2_000_000_000)
    run.exec_fused(); run.assemble(); p.check_status()
    for g, got, want in zip(w.gemms, run.results(), ref):
        assert np.array_equal(got.astype(np.float64), want), g.name


def test_blocks_of_odd_granule_counts_share_cta_pairs():
    """Uniform grid whose blocks are 416 (fwd, dgrad) or 192 (wgrad) rows high, i.e. an odd number of
    128-row half-tiles plus a ragged one: half-tiles of neighbouring blocks run as one pair, full and
    ragged, in every operand layout."""
    gemms, tensors = ci.projection_gemms(1664, [("p", 768, 896)])
    w = ci.Workload("odd-granules", gemms, tensors, uniform=(4, 2, 2))
    ts = ci.make_tensors(w, integer=True)
    p, op = lib_plan_for(w), oracle_plan_for(w)
    assert np.array_equal(task_matrix_lib(p), task_matrix_oracle(op))
    half_tiles = sum(p.task_num_tiles(i) for i in range(p.num_tasks))
    assert p.num_tiles < 0.6 * half_tiles                  # nearly every half-tile found a partner
    A, B = oracle_operands(w, ts)
    ref = nm.assemble(op, nm.execute(op, A, B))
    run = GpuRun(w, ts, p)
    run.exec_fused(); run.assemble(); p.check_status()
    for g, got, want in zip(w.gemms, run.results(), ref):
        assert np.array_equal(got.astype(np.float64), want), g.name


def test_row_granule_256_plan():
    """The planner option the first version of the kernel preferred (blocks of whole 256-row tiles)."""
    w = ci.config(3, 8)
    ts = ci.make_tensors(w, integer=True)
    p, op = lib_plan_for(w, gran_m=256), oracle_plan_for(w, gran_m=256)
    assert np.array_equal(task_matrix_lib(p), task_matrix_oracle(op))
    A, B = oracle_operands(w, ts)
    ref = nm.assemble(op, nm.execute(op, A, B))
    run = GpuRun(w, ts, p)
    run.exec_fused(); run.assemble(); p.check_status()
    for g, got, want in zip(w.gemms, run.results(), ref):
        assert np.array_equal(got.astype(np.float64), want), g.name


def test_short_pairs_straight_to_c_with_dropped_tasks():
    """Pairs of one to four K-blocks (attention-shaped GEMMs: the scheduler takes their tickets four at
    a time) whose blocks go straight to C as bulk stores: exact against the oracle on integer inputs.
    With one task of every second GEMM dropped, pairs that have nothing to run are skipped inside a batch of
    tickets, the bookkeeping names exactly the missing tasks, and the reissue completes C to the same bits."""
    w = ci.config(6, 4)                                  # 64 heads: K = 64 (scores) and K = 256 (context)
    ts = ci.make_tensors(w, integer=True)
    p, op = lib_plan_for(w), oracle_plan_for(w)
    A, B = oracle_operands(w, ts)
    ref = nm.assemble(op, nm.execute(op, A, B))
    run = GpuRun(w, ts, p)
    run.exec_opts(direct=True, finish=True); run.assemble(); p.check_status()
    good = run.results()
    for gi, g in enumerate(w.gemms):
        assert np.array_equal(good[gi].astype(np.float64), ref[gi]), g.name
    done = p.done_counts()
    assert all(done[i] == p.task_num_tiles(i) for i in range(p.num_tasks))

    p2 = lib_plan_for(w)
    t = p2.tasks()
    # the first task of every second GEMM that runs on at least two devices (its owner is lost for that GEMM;
    # the others survive and take the replacement pieces)
    failed = np.array([int(t[t["gemm"] == gi]["id"][0]) for gi in range(0, len(w.gemms), 2)
                       if len(set(t[t["gemm"] == gi]["dev"].tolist())) >= 2], dtype=np.uint32)
    assert len(failed) >= len(w.gemms) // 4
    p2.set_drops(failed)
    run2 = GpuRun(w, ts, p2)
    run2.exec_opts(direct=True, finish=True); run2.assemble()
    assert p2.status() == -9
    lost = set(failed.tolist())
    done = p2.done_counts()
    assert all((done[i] == 0) == (i in lost) for i in range(p2.num_tasks))
    run2.reissue(failed); run2.assemble()
    assert p2.status() == 0
    for g, a, b in zip(w.gemms, good, run2.results()):
        assert np.array_equal(a.view(np.uint32), b.view(np.uint32)), g.name
