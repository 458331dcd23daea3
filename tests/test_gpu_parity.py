"""Parity of the CUDA path against the oracle, through the C ABI.  Needs a B200."""
import numpy as np
import pytest

import cleave_inputs as ci
from helpers import (GpuRun, assert_within_tolerance, lib_plan_for, oracle_operands, oracle_plan_for,
                     task_matrix_lib, task_matrix_oracle)
from oracle import check, numerics as nm
from oracle.reissue import reissue as oracle_reissue

pytestmark = pytest.mark.gpu


def _custom_workload(tokens, projections, passes=("fwd", "dgrad", "wgrad"), n_devices=6, uniform=None, seed=0):
    gemms, tensors = ci.projection_gemms(tokens, projections, passes)
    return ci.Workload("custom", gemms, tensors, n_devices=n_devices, mem_range=(64 * ci.MB, 1 * ci.GB),
                       uniform=uniform, seed=seed)


def _run_and_compare_exact(w, opts=None, integer=True):
    opts = opts or {}
    ts = ci.make_tensors(w, integer=integer)
    p, op = lib_plan_for(w, **opts), oracle_plan_for(w, **opts)
    assert np.array_equal(task_matrix_lib(p), task_matrix_oracle(op))
    A, B = oracle_operands(w, ts)
    ref = nm.assemble(op, nm.execute(op, A, B))
    run = GpuRun(w, ts, p)
    run.exec()
    run.assemble()
    p.check_status()
    out = run.results()
    for gi, g in enumerate(w.gemms):
        if integer:
            assert np.array_equal(out[gi].astype(np.float64), ref[gi]), f"{g.name}: integer inputs must be exact"
        else:
            assert_within_tolerance(out[gi], ref[gi], nm.abs_bound(A[gi], B[gi]), what=g.name)
    done = p.done_counts()
    assert all(done[i] == p.task_num_tiles(i) for i in range(p.num_tasks))
    # the fused write-out (blocks of one-slice GEMMs straight to C, bulk stores where a chunk is whole and aligned,
    # K-split cells summed in the kernel) must give the same bits on the same plan
    fused = GpuRun(w, ts, p)
    fused.exec_opts(direct=True, finish=True)
    fused.assemble()
    p.check_status()
    for gi, g in enumerate(w.gemms):
        assert np.array_equal(out[gi].view(np.uint32), fused.results()[gi].view(np.uint32)), f"{g.name}: fused write-out differs"
    return p, op, run, ref


def test_config1_uniform_exact_and_gaussian():
    w = ci.config(1)
    _run_and_compare_exact(w, integer=True)
    _run_and_compare_exact(w, integer=False)


@pytest.mark.parametrize("passes", [("fwd",), ("dgrad",), ("wgrad",)])
def test_each_operand_layout_exact(passes):
    # several tiles per task, two K-slices, ragged last tile in every dimension
    w = _custom_workload(648, [("p", 456, 328)], passes=passes, n_devices=5)
    _run_and_compare_exact(w, dict(kslice_max=256))


def test_ragged_uniform_grid_exact():
    # block edges off the tile grid (multiples of 8 where the operand layout needs it, odd
    # elsewhere); K = 408 / 400 / 520 leave tails of 24 / 16 / 8 beyond a multiple of 64
    w = _custom_workload(520, [("p", 408, 400)], uniform=(3, 2, 1))
    w.n_devices = 0
    _run_and_compare_exact(w)


def test_wide_and_tall_tasks_exact():
    # one device: a single task per K-slice, many 128 x 256 tiles, three K-slices
    w = _custom_workload(1024, [("p", 832, 1280)], n_devices=1)
    p, *_ = _run_and_compare_exact(w, dict(kslice_max=512))
    assert max(p.ksplit(i) for i in range(3)) >= 2


@pytest.mark.parametrize("cfg,scale", [(2, 4), (3, 8), (5, 16)])
def test_scaled_configs_gaussian(cfg, scale):
    w = ci.config(cfg, scale)
    _run_and_compare_exact(w, integer=False)


def test_attention_gemms_as_tasks():
    """Many small independent GEMMs in one task list (scores Q.K^T and context P.V per head):
    every GEMM has its own operands and tensor maps; K = 64 is a single K-block."""
    w = ci.config(6, 4)                                  # 64 heads, seq 256, head dim 64: 128 GEMMs
    assert len(w.gemms) == 128
    _run_and_compare_exact(w, integer=True)
    p, *_ = _run_and_compare_exact(w, integer=False)
    assert p.num_tasks >= 2 * len(w.gemms)


def test_scaled_config2_integer_exact():
    _run_and_compare_exact(ci.config(2, 4), integer=True)


def test_churn_reissue_equals_no_failure():
    w = ci.config(4, 8)
    ts = ci.make_tensors(w, integer=False)
    p, op = lib_plan_for(w), oracle_plan_for(w)
    A, B = oracle_operands(w, ts)
    ref = nm.assemble(op, nm.execute(op, A, B))

    base = GpuRun(w, ts, p)                  # no failure
    base.exec(); base.assemble(); p.check_status()
    good = base.results()

    p2 = lib_plan_for(w)
    failed = ci.make_failed_ids(p2.num_tasks, w.fail_frac, w.seed + 2)
    p2.set_drops(failed)
    run = GpuRun(w, ts, p2)                  # arena poisoned with NaN: a skipped block stays NaN
    run.exec(); run.assemble()
    assert p2.status() == -9                 # E_INCOMPLETE: bookkeeping knows what is missing
    assert any(np.isnan(c).any() for c in run.results())
    done = p2.done_counts()
    assert all((done[i] == 0) == (i in set(failed.tolist())) for i in range(p2.num_tasks))

    run.reissue(failed)                      # explicit failed list
    new = oracle_reissue(op, failed)
    assert np.array_equal(task_matrix_lib(p2), task_matrix_oracle(op))
    run.assemble()
    assert p2.status() == 0
    out = run.results()
    for gi, g in enumerate(w.gemms):
        assert np.array_equal(out[gi], good[gi]), f"{g.name}: reissued result differs from the no-failure result"
        assert_within_tolerance(out[gi], ref[gi], nm.abs_bound(A[gi], B[gi]), what=g.name)

    # second wave, found by the bookkeeping itself (n = 0): drop some replacement tasks and re-run all
    again = [t.id for t in new[::4]]
    p2.set_drops(again)
    run.partials.fill_(float("nan"))
    run.exec(); run.assemble()
    assert p2.status() == -9
    run.reissue(None)
    oracle_reissue(op, again)
    assert np.array_equal(task_matrix_lib(p2), task_matrix_oracle(op))
    run.assemble()
    assert p2.status() == 0
    out = run.results()
    for gi in range(len(w.gemms)):
        assert np.array_equal(out[gi], good[gi])


def test_fused_write_out_equals_exec_plus_assemble():
    """One-slice GEMMs written straight to C by the exec kernel: same bits as the two-step path,
    also through a failure and its reissue."""
    import paper_2512_22142_b200 as cl
    w = ci.config(4, 8)
    ts = ci.make_tensors(w)
    p = lib_plan_for(w, kslice_max=512)
    S = [p.ksplit(i) for i in range(p.n_gemms)]
    assert 1 in S and max(S) > 1                      # both kinds of GEMM are present
    base = GpuRun(w, ts, p)
    base.exec(); base.assemble(); p.check_status()
    good = base.results()

    p2 = lib_plan_for(w, kslice_max=512)
    run = GpuRun(w, ts, p2)                            # C starts as NaN: nothing may be left unwritten
    launches_two_step = p2.num_launches
    run.exec_fused(); run.assemble(); p2.check_status()
    assert p2.num_launches < launches_two_step         # the one-slice groups are not launched any more
    for g, a, b in zip(w.gemms, good, run.results()):
        assert np.array_equal(a.view(np.uint32), b.view(np.uint32)), g.name

    import torch
    other = [torch.empty_like(c) for c in run.C]
    with pytest.raises(cl.CleaveError) as e:           # part of the result already sits in the first C
        p2.assemble(run.partials, other)
    assert e.value.code == -1

    failed = ci.make_failed_ids(p2.num_tasks, w.fail_frac, w.seed + 2)
    p2.set_drops(failed)
    for c in run.C:
        c.fill_(float("nan"))
    run.partials.fill_(float("nan"))
    run.exec_fused(); run.assemble()
    assert p2.status() == -9 and any(np.isnan(c).any() for c in run.results())
    run.reissue(failed); run.assemble()
    assert p2.status() == 0
    for g, a, b in zip(w.gemms, good, run.results()):
        assert np.array_equal(a.view(np.uint32), b.view(np.uint32)), g.name
    run.exec(); run.assemble(); p2.check_status()      # a plain exec ends fused mode
    for g, a, b in zip(w.gemms, good, run.results()):
        assert np.array_equal(a.view(np.uint32), b.view(np.uint32)), g.name


@pytest.mark.parametrize("S", [1, 2, 3, 4, 5, 8, 13])
def test_assembly_bit_exact_vs_fp32_tree(S):
    """Random fp32 partials (not products): the assembly kernel must reproduce the balanced
    pairwise tree bit for bit."""
    import torch
    w = _custom_workload(384, [("p", 128 * S, 320)], passes=("fwd",), n_devices=7, seed=S)
    opts = dict(ksplit=S, kslice_max=0, ksplit_cap=32)
    p, op = lib_plan_for(w, **opts), oracle_plan_for(w, **opts)
    assert p.ksplit(0) == S
    rng = np.random.default_rng(S)
    arena = (rng.standard_normal(op.arena_elems) * 10.0 ** rng.integers(-3, 4, op.arena_elems)).astype(np.float32)
    ref = nm.assemble(op, arena, dtype=np.float32)[0]
    g = w.gemms[0]
    C = torch.zeros((g.M, g.N), dtype=torch.float32, device="cuda:0")
    part = torch.from_numpy(arena).cuda()
    p.assemble(part, [C])
    assert p.status() == -9                  # nothing was executed: bookkeeping says incomplete ...
    out = C.cpu().numpy()
    assert np.array_equal(out.view(np.uint32), ref.view(np.uint32))   # ... the sums are exact all the same


def test_assembly_scalar_path_bit_exact():
    import torch
    gemms, tensors = ci.projection_gemms(50, [("p", 64, 45)], ("fwd",))      # N = 45: no float4 alignment
    w = ci.Workload("odd", gemms, tensors, uniform=(3, 2, 1))
    from oracle.plan import Opts, plan_uniform
    import paper_2512_22142_b200 as cl
    p = cl.plan_uniform(w.gemms, 3, 2, 1)
    op = oracle_plan_for(w)
    rng = np.random.default_rng(0)
    arena = rng.standard_normal(op.arena_elems).astype(np.float32)
    ref = nm.assemble(op, arena, dtype=np.float32)[0]
    C = torch.zeros((50, 45), dtype=torch.float32, device="cuda:0")
    p.assemble(torch.from_numpy(arena).cuda(), [C])
    torch.cuda.synchronize()
    assert np.array_equal(C.cpu().numpy().view(np.uint32), ref.view(np.uint32))


@pytest.mark.parametrize("T,din,dout", [(1, 8, 8), (8, 8, 8), (130, 72, 264), (257, 64, 8), (300, 520, 136)])
def test_degenerate_and_small_shapes_exact(T, din, dout):
    """Smallest legal shapes (one row, K = 8), shapes below one tile, and shapes one element past a
    tile edge, in all three operand layouts, as a single task and as a ragged 2 x 2 x 1 grid."""
    for grid in ((1, 1, 1), (2, 2, 1)):
        if grid[0] > min(T, din) or grid[1] > min(din, dout) or (grid != (1, 1, 1) and (din % 16 or dout % 16)):
            continue
        w = _custom_workload(T, [("p", din, dout)], uniform=grid)
        w.n_devices = 0
        _run_and_compare_exact(w)


def test_more_slices_than_granules_and_many_devices():
    # forced K-split larger than the number of K-granules is clamped; more devices than output cells
    w = _custom_workload(256, [("p", 128, 256)], n_devices=40)
    p, op, run, ref = _run_and_compare_exact(w, dict(ksplit=9))
    assert p.ksplit(0) == 1 and p.ksplit(2) == 2          # K = 128 -> 1 granule; K = 256 -> 2 granules


def test_bad_arguments_are_rejected_on_the_host():
    import torch
    import paper_2512_22142_b200 as cl
    w = ci.config(1)
    p = lib_plan_for(w)
    x = torch.zeros(256, 768, dtype=torch.bfloat16, device="cuda:0")
    wt = torch.zeros(768, 768, dtype=torch.bfloat16, device="cuda:0")
    part = torch.zeros(p.arena_elems + 64, dtype=torch.float32, device="cuda:0")
    c = torch.zeros(256, 768, dtype=torch.float32, device="cuda:0")
    for bad in (lambda: p.exec([x.data_ptr() + 2], [wt], part),            # operand not 16-byte aligned
                lambda: p.exec([0], [wt], part),                           # null operand
                lambda: p.exec([x], [wt], part[1:]),                       # arena not 128-byte aligned
                lambda: p.assemble(part, [c.data_ptr() + 4]),              # C not 16-byte aligned
                lambda: p.reissue([99], [x], [wt], part)):                 # task id out of range
        with pytest.raises(cl.CleaveError) as e:
            bad()
        assert e.value.code in (-1, -5)
    p.exec([x], [wt], part); p.assemble(part, [c]); p.check_status()       # the plan is still usable afterwards


def test_new_operand_buffers_and_side_stream():
    """The same plan run on other operand buffers (the tensor maps must follow the pointers) and on
    a stream other than the default one."""
    import torch
    w = ci.config(2, 8)
    p, op = lib_plan_for(w), oracle_plan_for(w)
    side = torch.cuda.Stream()
    for seed in (0, 1):
        ts = ci.make_tensors(w, seed=seed, integer=True)
        A, B = oracle_operands(w, ts)
        ref = nm.assemble(op, nm.execute(op, A, B))
        run = GpuRun(w, ts, p)                           # fresh device tensors: new addresses
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            run.exec_fused(); run.assemble()
        side.synchronize()
        p.check_status()
        for g, got, want in zip(w.gemms, run.results(), ref):
            assert np.array_equal(got.astype(np.float64), want), (seed, g.name)


def test_every_task_dropped():
    """Nothing to run: the kernel's scheduler finds no runnable tile, the bookkeeping reports every
    task unfinished, and with every device dead no re-plan exists."""
    import paper_2512_22142_b200 as cl
    w = ci.config(2, 8)
    ts = ci.make_tensors(w)
    p = lib_plan_for(w)
    p.set_drops(np.arange(p.num_tasks))
    run = GpuRun(w, ts, p)
    run.exec(); run.assemble()
    assert p.status() == -9 and p.done_counts().sum() == 0
    assert all(np.isnan(c).all() for c in run.results())
    with pytest.raises(cl.CleaveError) as e:
        run.reissue(None)
    assert e.value.code == -4                             # E_NO_DEVICES
    p.set_drops([])
    run.exec(); run.assemble(); p.check_status()
    assert all(np.isfinite(c).all() for c in run.results())


def test_plans_off_the_alignment_rules_run_on_the_plain_kernel():
    """K-ranges that do not start on multiples of 64, leading dimensions that are no multiples of 8,
    blocks that start on odd rows and columns: the tensor-core kernel cannot take such plans, the plain
    kernel runs them -- same blocks, same bookkeeping, same churn path -- in all three layouts."""
    import torch
    gemms, tensors = ci.projection_gemms(90, [("p", 200, 84)])              # K = 200 in 2 slices of 100; N = 84; M = 90
    w = ci.Workload("off-rules", gemms, tensors, uniform=(3, 2, 2))
    ts = ci.make_tensors(w, integer=True)
    p, op = lib_plan_for(w), oracle_plan_for(w)
    assert np.array_equal(task_matrix_lib(p), task_matrix_oracle(op))
    A, B = oracle_operands(w, ts)
    ref = nm.assemble(op, nm.execute(op, A, B))
    run = GpuRun(w, ts, p)
    run.exec_fused(); run.assemble(); p.check_status()                      # a fused call falls back to two steps
    for g, got, want in zip(w.gemms, run.results(), ref):
        assert np.array_equal(got.astype(np.float64), want), g.name
    done = p.done_counts()
    assert all(done[i] == p.task_num_tiles(i) for i in range(p.num_tasks))
    # churn on the same path
    failed = np.array([1, 7, 20], dtype=np.uint32)
    p.set_drops(failed)
    run.partials.fill_(float("nan"))
    for c in run.C:
        c.fill_(float("nan"))
    run.exec(); run.assemble()
    assert p.status() == -9 and (p.done_counts()[failed] == 0).all()
    run.reissue(None)
    oracle_reissue(op, failed)
    assert np.array_equal(task_matrix_lib(p), task_matrix_oracle(op))
    run.assemble()
    assert p.status() == 0
    for g, got, want in zip(w.gemms, run.results(), ref):
        assert np.array_equal(got.astype(np.float64), want), g.name
    # Gaussian inputs within the path's tolerance
    ts = ci.make_tensors(w)
    A, B = oracle_operands(w, ts)
    p2, op2 = lib_plan_for(w), oracle_plan_for(w)
    ref = nm.assemble(op2, nm.execute(op2, A, B))
    run2 = GpuRun(w, ts, p2)
    run2.exec(); run2.assemble(); p2.check_status()
    for gi, (g, got, want) in enumerate(zip(w.gemms, run2.results(), ref)):
        assert_within_tolerance(got, want, nm.abs_bound(A[gi], B[gi]), what=g.name)
