"""Host side of the library, no GPU: the C-ABI library loads and exports what the header
declares; its planner and churn re-planner reproduce the oracle's task lists exactly; host-side
error codes."""
import os
import re

import numpy as np
import pytest

import cleave_inputs as ci
from helpers import (lib_plan_for, oracle_gemms, oracle_plan_for, task_matrix_lib, task_matrix_oracle)
from oracle.cost import devices_from_array
from oracle.plan import Gemm, Opts, plan as oracle_plan, plan_uniform as oracle_plan_uniform, PlanError
from oracle.reissue import reissue as oracle_reissue

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def cl():
    from paper_2512_22142_b200.build import build_library
    build_library()
    import paper_2512_22142_b200 as cl
    return cl


def test_every_declared_symbol_is_exported(cl):
    header = open(os.path.join(ROOT, "include", "cleave.h")).read()
    declared = set(re.findall(r"^CLEAVE_API [^;(]*?\b(cleave_\w+)\(", header, flags=re.M))
    assert len(declared) >= 20
    for name in declared:
        assert hasattr(cl.lib, name), name
    assert cl.strerror(0) == "ok" and "unknown" not in cl.strerror(-9)


@pytest.mark.parametrize("cfg,scale", [(1, 1), (2, 1), (2, 4), (3, 4), (3, 1), (5, 8), (5, 1)])
def test_planner_equals_oracle(cl, cfg, scale):
    w = ci.config(cfg, scale)
    p, op = lib_plan_for(w), oracle_plan_for(w)
    assert np.array_equal(task_matrix_lib(p), task_matrix_oracle(op))
    assert p.arena_elems == op.arena_elems and p.num_original == len(op.tasks)
    for gi in range(len(w.gemms)):
        assert p.ksplit(gi) == op.ksplit[gi]
        assert p.makespan_ns(gi) == op.makespan_ns[gi]
        assert p.tstar_ns(gi) == op.t_star[gi]


@pytest.mark.parametrize("alpha_milli,beta_ppm", [(3000, 50_000), (1500, 10_000), (2500, 200_000)])
def test_tail_aware_planner_equals_oracle(cl, alpha_milli, beta_ppm):
    """Appendix C's tail-aware cost (latencies at their CVaR): same task lists, and levels of a DAG
    cost what the oracle's level recursion says."""
    from oracle.levels import plan_level_costs
    w = ci.config(3, 4)
    kw = dict(tail_alpha_milli=alpha_milli, tail_beta_ppm=beta_ppm)
    p, op = lib_plan_for(w, **kw), oracle_plan_for(w, **kw)
    assert np.array_equal(task_matrix_lib(p), task_matrix_oracle(op))
    base = lib_plan_for(w)
    assert all(p.tstar_ns(i) == op.t_star[i] and p.tstar_ns(i) > base.tstar_ns(i) for i in range(p.n_gemms))
    gemms, tensors, produced = ci.two_branch_chain(512, 256, 384, 256)
    wc = ci.Workload("chain", gemms, tensors, n_devices=9, mem_range=(64 * ci.MB, ci.GB), produced=produced)
    pc, oc = lib_plan_for(wc, **kw), oracle_plan_for(wc, **kw)
    assert np.array_equal(task_matrix_lib(pc), task_matrix_oracle(oc))
    want = plan_level_costs(oc, [g.level for g in gemms])
    assert pc.num_levels == 3 and pc.step_makespan_ns == want[-1]
    assert [pc.level_makespan_ns(s) for s in range(3)] == [want[0], want[1] - want[0], want[2] - want[1]]
    with pytest.raises(cl.CleaveError) as e:
        lib_plan_for(w, tail_alpha_milli=1000)              # infinite mean: no CVaR
    assert e.value.code == -1


@pytest.mark.parametrize("seed", range(10))
def test_planner_equals_oracle_random_small(cl, seed):
    rng = np.random.default_rng(100 + seed)
    gemms = [Gemm(int(rng.integers(1, 900)), int(rng.integers(1, 900)), int(rng.integers(1, 3000)),
                  int(rng.integers(0, 2)), int(rng.integers(0, 2))) for _ in range(3)]
    devs = ci.make_devices(int(rng.integers(1, 60)), 1 << int(rng.integers(16, 22)), 1 << 26, seed)
    kw = dict(gran_m=int(rng.choice([16, 32, 64])), gran_n=int(rng.choice([16, 32, 64])), gran_k=int(rng.choice([32, 64])),
              kslice_max=int(rng.choice([0, 256, 1024])), ksplit=int(rng.choice([0, 0, 2, 5])), ksplit_cap=int(rng.choice([2, 8])))

    class G:  # the binding wants lda / ldb as well
        def __init__(self, g):
            self.M, self.N, self.K, self.transA, self.transB = g.M, g.N, g.K, g.transA, g.transB
            self.lda = g.M if g.transA else g.K
            self.ldb = g.K if g.transB else g.N
    try:
        op = oracle_plan(gemms, devices_from_array(devs), Opts(**kw))
    except PlanError as e:
        with pytest.raises(cl.CleaveError) as ce:
            cl.plan([G(g) for g in gemms], devs, cl.default_opts(**kw))
        assert cl.strerror(ce.value.code).startswith("no plan") == (e.code == "E_INFEASIBLE")
        return
    p = cl.plan([G(g) for g in gemms], devs, cl.default_opts(**kw))
    assert np.array_equal(task_matrix_lib(p), task_matrix_oracle(op))


@pytest.mark.parametrize("cfg,scale", [(4, 8), (4, 2), (4, 1)])
def test_replan_equals_oracle(cl, cfg, scale):
    w = ci.config(cfg, scale)
    p, op = lib_plan_for(w), oracle_plan_for(w)
    failed = ci.make_failed_ids(p.num_tasks, w.fail_frac, w.seed + 2)
    assert len(failed) == round(0.1 * p.num_tasks)
    first = p.replan(failed)
    new = oracle_reissue(op, failed)
    assert first == new[0].id == p.num_original
    assert np.array_equal(task_matrix_lib(p), task_matrix_oracle(op))
    # a second wave hits some of the replacement tasks and some survivors
    wave2 = np.unique(np.concatenate([np.arange(first, p.num_tasks, 5),
                                      [t.id for t in op.tasks[:first:97] if not (t.flags & 1)]])).astype(np.uint32)
    p.replan(wave2)
    oracle_reissue(op, wave2)
    assert np.array_equal(task_matrix_lib(p), task_matrix_oracle(op))
    with pytest.raises(cl.CleaveError) as e:
        p.replan(failed[:1])
    assert e.value.code == -1                                    # already superseded
    with pytest.raises(cl.CleaveError) as e:
        p.replan([p.num_tasks])
    assert e.value.code == -5


def test_uniform_and_errors(cl):
    w = ci.config(1)
    p = cl.plan_uniform(w.gemms, 4, 4, 2)
    t = p.tasks()
    assert p.num_tasks == 32 and p.arena_elems == 393216 and p.num_tiles == 16   # two 64-row blocks of a column share a pair of CTAs
    assert set(zip(t["m1"] - t["m0"], t["n1"] - t["n0"], t["k1"] - t["k0"])) == {(64, 192, 384)}
    with pytest.raises(cl.CleaveError) as e:
        p.set_drops([32])
    assert e.value.code == -5                                    # E_RANGE
    p.set_drops([0, 31])
    p.set_drops([])
    with pytest.raises(cl.CleaveError) as e:
        cl.plan_uniform(w.gemms, 0, 4, 2)
    assert e.value.code == -1                                    # E_INVAL
    with pytest.raises(cl.CleaveError) as e:
        cl.plan(w.gemms, np.zeros((0, 6), dtype=np.uint64))
    assert e.value.code == -4                                    # E_NO_DEVICES
    tiny = ci.make_devices(4, 1 << 10, 1 << 11, 0)               # 1-2 KB of memory: nothing fits
    with pytest.raises(cl.CleaveError) as e:
        cl.plan(w.gemms, tiny)
    assert e.value.code == -3                                    # E_INFEASIBLE


def test_header_is_plain_c_and_defaults_agree_with_oracle(cl, tmp_path):
    import subprocess
    src = tmp_path / "use_header.c"
    src.write_text('#include "cleave.h"\nint main(void) { cleave_plan_opts_t o; cleave_task_t t; (void)o; (void)t; '
                   'return sizeof(cleave_task_t) == 64 && sizeof(cleave_device_t) == 48 && sizeof(cleave_gemm_t) == 24 ? 0 : 1; }\n')
    exe = tmp_path / "use_header"
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Werror", "-I", os.path.join(ROOT, "include"), str(src), "-o", str(exe)], check=True)
    assert subprocess.run([str(exe)]).returncode == 0
    o, ref = cl.default_opts(), Opts()
    for name in ("gran_m", "gran_n", "gran_k", "kslice_max", "ksplit", "ksplit_cap", "reissue_fanout", "b_in", "b_out", "tail_alpha_milli", "tail_beta_ppm"):
        assert getattr(o, name) == getattr(ref, name), name


def test_levels_and_new_options_on_the_host(cl):
    """DAG levels, the finishable flag and argument checks that need no device."""
    from oracle.levels import plan_level_costs
    gemms, tensors, produced = ci.two_branch_chain(512, 256, 384, 256)
    w = ci.Workload("chain", gemms, tensors, n_devices=7, mem_range=(64 * ci.MB, ci.GB), produced=produced)
    p, op = lib_plan_for(w, kslice_max=256), oracle_plan_for(w, kslice_max=256)
    assert np.array_equal(task_matrix_lib(p), task_matrix_oracle(op))
    assert p.num_levels == 3
    want = plan_level_costs(op, [g.level for g in gemms])
    assert p.step_makespan_ns == want[-1] and p.level_makespan_ns(0) == want[0] and p.level_makespan_ns(7) == 0
    # on the 128-grid every K-split GEMM can be summed by the exec kernel; one-slice GEMMs have nothing to sum
    for i in range(p.n_gemms):
        assert p.finishable(i) == (p.ksplit(i) >= 2)
    assert not p.finishable(99)
    # more than 8 K-slices, or N not a multiple of 4, are left to the assembly kernel
    g1, t1 = ci.projection_gemms(256, [("p", 2048, 256)], ("fwd",))
    many = cl.plan(g1, ci.make_devices(4, 64 * ci.MB, ci.GB, 0), cl.default_opts(ksplit=12, kslice_max=0, ksplit_cap=32))
    assert many.ksplit(0) == 12 and not many.finishable(0)
    # levels beyond the limit are refused when the plan is made
    class G:
        def __init__(self, g, level):
            self.__dict__.update(M=g.M, N=g.N, K=g.K, transA=g.transA, transB=g.transB, lda=g.lda, ldb=g.ldb, level=level)
    with pytest.raises(cl.CleaveError) as e:
        cl.plan([G(g1[0], 4096)], ci.make_devices(4, 64 * ci.MB, ci.GB, 0))
    assert e.value.code == -1
    ok = cl.plan([G(g1[0], 4095)], ci.make_devices(4, 64 * ci.MB, ci.GB, 0))
    assert ok.num_levels == 4096
    # tile counts: a plan on the 128-grid is cut into full 256 x 256 pairs per K-range, whatever its blocks
    w3 = ci.config(3, 4)
    p3 = lib_plan_for(w3)
    pairs = sum(-(-g.M // 256) * -(-g.N // 256) * p3.ksplit(i) for i, g in enumerate(w3.gemms))
    assert p3.num_tiles == pairs
    quadrants = sum(p3.task_num_tiles(i) for i in range(p3.num_tasks))
    assert quadrants == sum(-(-g.M // 128) * -(-g.N // 128) * p3.ksplit(i) for i, g in enumerate(w3.gemms))
