"""Pins of the churn re-planner (Section 4.2): survivors fixed, dead devices excluded, failed
rectangles covered exactly once, the cache-aware downlink term, and the end result unchanged."""
import copy

import numpy as np
import pytest

import cleave_inputs as ci
from oracle import check, numerics as nm
from oracle.cost import c_comp, c_dl, c_ul, devices_from_array
from oracle.plan import (FLAG_REISSUED, FLAG_SUPERSEDED, UNIFORM_DEVICE, Gemm, Opts, PlanError,
                         plan, plan_uniform)
from oracle.reissue import reissue, recovery_makespan_ns


def test_cache_aware_owner_choice():
    # 2 x 2 grid, one slice; task 0 (rows 0:8, cols 0:24) fails.  Device 1 caches its rows,
    # device 2 its columns, device 3 nothing.  All devices are identical, so the owner is the
    # one that has the longer side cached: device 2 (24 columns > 8 rows).
    p = plan_uniform([Gemm(16, 48, 32)], 2, 2, 1, Opts(gran_m=8, gran_n=8, gran_k=8, reissue_fanout=1))
    new = reissue(p, [0])
    assert len(new) == 1
    t = new[0]
    assert t.dev == 2 and t.parent == 0 and t.flags == FLAG_REISSUED and t.id == 4
    d = UNIFORM_DEVICE
    expect = max(c_dl(8, 0, 32, d, 2, latency=False), c_ul(8, 24, d, 4), c_comp(8, 24, 32, d))
    assert t.cost_ns == expect
    assert p.tasks[0].flags & FLAG_SUPERSEDED and p.dead[0] == {0}
    assert recovery_makespan_ns(p, new) == expect


def test_pieces_and_lpt_spread():
    p = plan_uniform([Gemm(64, 32, 16)], 1, 4, 1, Opts(gran_m=8, gran_n=8, gran_k=8, reissue_fanout=4))
    before = copy.deepcopy(p.tasks)
    new = reissue(p, [1])
    assert [(t.m0, t.m1) for t in new] == [(0, 16), (16, 32), (32, 48), (48, 64)]
    assert all((t.n0, t.n1, t.k0, t.k1) == (8, 16, 0, 16) for t in new)
    assert [t.part_off for t in new] == [before[1].part_off + r * 8 for r in (0, 16, 32, 48)]
    assert 1 not in {t.dev for t in new}                 # the dead device gets nothing
    assert len({t.dev for t in new}) == 3                # spread over all three survivors
    for a, b in zip(before, p.tasks):                    # survivors' assignments stay fixed
        if a.id != 1:
            assert a.astuple() == b.astuple()
    check.check_cover(p, 0)
    check.check_arena(p)
    assert (check.cover_count_bruteforce(p, 0) == 1).all()


def test_errors():
    p = plan_uniform([Gemm(16, 16, 16)], 2, 1, 1, Opts(gran_m=8, gran_n=8, gran_k=8))
    with pytest.raises(PlanError) as e:
        reissue(p, [2])
    assert e.value.code == "E_RANGE"
    with pytest.raises(PlanError) as e:
        reissue(p, [0, 1])
    assert e.value.code == "E_NO_DEVICES"
    reissue(p, [0])
    with pytest.raises(PlanError) as e:
        reissue(p, [0])
    assert e.value.code == "E_INVAL"
    assert reissue(p, []) == []


@pytest.mark.parametrize("seed", range(4))
def test_reissue_result_equals_no_failure(seed):
    w = ci.config(4, scale=16)
    devs = devices_from_array(ci.workload_devices(w))
    gemms = [Gemm(g.M, g.N, g.K, g.transA, g.transB) for g in w.gemms]
    o = Opts(gran_m=32, gran_n=32, gran_k=32, kslice_max=128)
    p = plan(gemms, devs, o)
    ts = ci.make_tensors(w, seed=seed, integer=True)
    A = [nm.op_a(nm.bf16_bits_to_f64(ci.bf16_bits(ts[g.a_key])), g.transA) for g in w.gemms]
    B = [nm.op_b(nm.bf16_bits_to_f64(ci.bf16_bits(ts[g.b_key])), g.transB) for g in w.gemms]
    ref = nm.assemble(p, nm.execute(p, A, B))
    for gi in range(len(gemms)):
        assert np.array_equal(ref[gi], A[gi] @ B[gi])

    failed = ci.make_failed_ids(len(p.tasks), w.fail_frac, w.seed + 2 + seed)
    assert len(failed) > 0
    arena = nm.execute(p, A, B, dropped=failed)
    assert any(np.isnan(c).any() for c in nm.assemble(p, arena))
    n0 = len(p.tasks)
    new = reissue(p, failed)
    dead_owner = {(p.tasks[f].gemm, p.tasks[f].dev) for f in failed}
    assert all((t.gemm, t.dev) not in dead_owner for t in new)
    for gi in range(len(gemms)):
        check.check_cover(p, gi)
    check.check_constraints(p)
    check.check_arena(p)
    nm.execute(p, A, B, task_ids=range(n0, len(p.tasks)), arena=arena)
    out = nm.assemble(p, arena)
    for gi in range(len(gemms)):
        assert np.array_equal(out[gi], ref[gi])

    # second wave: some replacement pieces fail too
    again = [t.id for t in new[::3]]
    arena2 = nm.execute(p, A, B, dropped=list(failed) + again)
    n1 = len(p.tasks)
    reissue(p, again)
    nm.execute(p, A, B, task_ids=range(n1, len(p.tasks)), arena=arena2)
    check.check_arena(p)
    out = nm.assemble(p, arena2)
    for gi in range(len(gemms)):
        check.check_cover(p, gi)
        assert np.array_equal(out[gi], ref[gi])
