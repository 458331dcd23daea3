"""Pins of the oracle planner against what the paper fixes: exact coverage, the zero-task and
memory constraints, special cases with a known answer, and the Eq. 18 lower bound."""
import numpy as np
import pytest

import cleave_inputs as ci
from oracle import check
from oracle.cost import Device, devices_from_array, lower_bound_ns, task_mem
from oracle.plan import (Gemm, Opts, PlanError, apportion, capacity, plan, plan_uniform, r_mem,
                         split_counts)


def small_devices(n, seed, mem_lo=1 << 20, mem_hi=1 << 24):
    return devices_from_array(ci.make_devices(n, mem_lo, mem_hi, seed))


def test_uniform_config1_matches_stated_geometry():
    # Config 1: 256x768x768 in a 4x4 grid x 2 K-slices -> 32 tasks of 64x192x384
    p = plan_uniform([Gemm(256, 768, 768)], 4, 4, 2)
    assert len(p.tasks) == 32 and p.arena_elems == 393216
    for t in p.tasks:
        assert (t.alpha, t.beta, t.kappa) == (64, 192, 384)
        assert t.part_off == t.id * 12288 and t.dev == t.id and t.parent == t.id
    # ids: block-row-major, then slice
    t = p.tasks[2 * (1 * 4 + 2) + 1]
    assert (t.m0, t.n0, t.k0, t.kslice) == (64, 384, 384, 1)
    check.check_cover(p, 0)
    assert (check.cover_count_bruteforce(p, 0) == 1).all()


@pytest.mark.parametrize("M,N,K,gm,gn,gk", [(7, 5, 9, 3, 2, 4), (10, 11, 3, 1, 1, 1), (1, 1, 1, 1, 1, 1)])
def test_uniform_ragged_cover(M, N, K, gm, gn, gk):
    p = plan_uniform([Gemm(M, N, K)], gm, gn, gk)
    assert (check.cover_count_bruteforce(p, 0) == 1).all()
    assert sum(t.alpha * t.beta * t.kappa for t in p.tasks) == M * N * K


@pytest.mark.parametrize("seed", range(12))
def test_planned_cover_bruteforce_tiny(seed):
    rng = np.random.default_rng(seed)
    M, N, K = (int(x) for x in rng.integers(1, 40, 3))
    D = int(rng.integers(1, 24))
    o = Opts(gran_m=int(rng.integers(1, 6)), gran_n=int(rng.integers(1, 6)), gran_k=int(rng.integers(1, 6)),
             kslice_max=int(rng.choice([0, 4, 16])), ksplit=int(rng.choice([0, 0, 1, 2, 3])))
    p = plan([Gemm(M, N, K)], small_devices(D, seed), o)
    cnt = check.cover_count_bruteforce(p, 0)
    assert cnt.min() == 1 and cnt.max() == 1          # every (i, j, k) exactly once
    check.check_cover(p, 0)
    check.check_constraints(p)
    check.check_arena(p)
    assert sum(t.alpha * t.beta for t in p.tasks) == p.ksplit[0] * M * N


def test_single_slice_is_the_papers_formulation():
    # kslice_max = 0 and D <= cells: every task spans the full inner dimension, and the areas add up to m*q
    devs = small_devices(9, 3, 1 << 26, 1 << 28)
    p = plan([Gemm(512, 384, 640)], devs, Opts(gran_m=64, gran_n=64, gran_k=64, kslice_max=0))
    assert p.ksplit == [1]
    assert all((t.k0, t.k1) == (0, 640) for t in p.tasks)
    assert sum(t.alpha * t.beta for t in p.tasks) == 512 * 384
    owners = [t.dev for t in p.tasks]
    assert len(owners) == len(set(owners))            # one shard per device


def test_homogeneous_devices_give_equal_grid():
    # 16 identical devices, Mg = Ng = 8 (granule 128), S = 1 -> 4 x 4 grid of equal 256 x 256 blocks
    devs = devices_from_array(ci.homogeneous_devices(16))
    p = plan([Gemm(1024, 1024, 512)], devs, Opts(gran_m=128, gran_n=128, kslice_max=0))
    assert len(p.tasks) == 16
    assert {(t.alpha, t.beta, t.kappa) for t in p.tasks} == {(256, 256, 512)}
    assert {(t.m0, t.n0) for t in p.tasks} == {(i * 256, j * 256) for i in range(4) for j in range(4)}
    assert len({t.cost_ns for t in p.tasks}) == 1


def test_zero_task_rule_excludes_straggler():
    fast = Device(1 << 30, 20_000_000, 100_000_000, 50_000_000, 1000, 1000)
    slow = Device(1 << 30, 20_000_000, 1_000, 1_000, 1000, 1000)      # 1 kB/s links
    p = plan([Gemm(512, 512, 256)], [fast, slow, fast, fast], Opts(kslice_max=0))
    assert 1 not in {t.dev for t in p.tasks}
    check.check_cover(p, 0)


def test_more_capable_devices_get_more_area():
    devs = small_devices(32, 7, 1 << 28, 1 << 30)
    g = Gemm(4096, 4096, 1024)
    p = plan([g], devs, Opts(kslice_max=0))
    caps = [capacity(d, p.t_star[0], 1024, p.opts) for d in devs]
    area = {}
    for t in p.tasks:
        area[t.dev] = area.get(t.dev, 0) + t.alpha * t.beta
    best, worst = max(area, key=lambda k: caps[k]), min(area, key=lambda k: caps[k])
    assert area[best] >= area[worst]
    # areas correlate with capability (workload proportional to capability, Appendix B)
    ks = sorted(area)
    r = np.corrcoef([caps[k] for k in ks], [area[k] for k in ks])[0, 1]
    assert r > 0.8


def test_memory_repair_and_infeasible():
    o = Opts(gran_m=16, gran_n=16, gran_k=16, kslice_max=0)
    # One granule row, eight granule columns, two devices: each share is a 16 x 64 strip whose
    # footprint (16+64)*64*2 + 16*64*4 = 14336 B exceeds a 13000 B budget although a square block
    # of the same area would fit -> the strip is cut in two 16 x 32 tasks on the same device.
    devs = [Device(13000, 10_000_000, 10 ** 8, 10 ** 8, 0, 0)] * 2
    p = plan([Gemm(16, 128, 64)], devs, o)
    assert len(p.tasks) == 4 and {(t.alpha, t.beta) for t in p.tasks} == {(16, 32)}
    assert [t.dev for t in p.tasks] == [p.tasks[0].dev] * 2 + [p.tasks[2].dev] * 2
    check.check_cover(p, 0)
    check.check_constraints(p)
    check.check_arena(p)
    cell = task_mem(16, 16, 64, 2, 4)
    with pytest.raises(PlanError) as e:
        plan([Gemm(64, 64, 64)], [Device(cell - 1, 10_000_000, 10 ** 8, 10 ** 8, 0, 0)] * 4, o)
    assert e.value.code == "E_INFEASIBLE"
    with pytest.raises(PlanError) as e:
        plan([Gemm(64, 64, 64)], [], o)
    assert e.value.code == "E_NO_DEVICES"


def test_auto_ksplit():
    devs = small_devices(8, 1, 1 << 28, 1 << 30)
    assert plan([Gemm(512, 256, 8192)], devs[:4], Opts()).ksplit == [2]        # depth cap 4096
    assert plan([Gemm(512, 256, 11008)], devs[:4], Opts()).ksplit == [3]
    assert plan([Gemm(512, 256, 4096)], devs[:4], Opts()).ksplit == [1]
    assert plan([Gemm(512, 256, 4096)], devs[:4], Opts(kslice_max=2048)).ksplit == [2]
    # more devices than output cells -> split K so that all can work (2x2 cells, 8 devices)
    assert plan([Gemm(512, 256, 512)], devs, Opts()).ksplit == [2]
    # K-slices are consecutive, granule aligned, sizes differ by at most one granule
    p = plan([Gemm(512, 256, 11008)], devs[:4], Opts())
    ranges = sorted({(t.k0, t.k1) for t in p.tasks})
    assert ranges == [(0, 3712), (3712, 7424), (7424, 11008)]


def test_makespan_respects_lower_bound():
    for cfg, scale in ((2, 4), (3, 8)):
        w = ci.config(cfg, scale=scale)
        devs = devices_from_array(ci.workload_devices(w))
        gemms = [Gemm(g.M, g.N, g.K, g.transA, g.transB) for g in w.gemms]
        p = plan(gemms, devs, Opts())
        for gi, g in enumerate(gemms):
            check.check_cover(p, gi)
            assert p.makespan_ns[gi] >= lower_bound_ns(2 * g.M * g.N * g.K, devs)   # Eq. 18, first term
        check.check_constraints(p)
        check.check_arena(p)


def test_helpers():
    assert apportion(10, [1, 1, 1]) == [4, 3, 3]
    assert apportion(3, [5, 1, 1]) == [1, 1, 1]
    assert apportion(12, [6, 3, 0]) == [7, 4, 1]
    assert sum(apportion(97, [13, 7, 29, 5])) == 97
    assert split_counts(11, 3) == [4, 4, 3]
    r = r_mem(10 ** 6, 100, 2, 4)
    assert 2 * r * 100 * 2 + r * r * 4 <= 10 ** 6 < 2 * (r + 1) * 100 * 2 + (r + 1) ** 2 * 4


def _guillotine_partitions(r0, r1, c0, c1, max_parts):
    """All ways to cut the granule rectangle [r0,r1) x [c0,c1) into at most max_parts rectangles by
    recursive straight cuts (every exact tiling of so small a grid is of this kind)."""
    out = [[(r0, r1, c0, c1)]]
    if max_parts < 2:
        return out
    for cut in range(r0 + 1, r1):
        for k in range(1, max_parts):
            for a in _guillotine_partitions(r0, cut, c0, c1, k):
                for b in _guillotine_partitions(cut, r1, c0, c1, max_parts - len(a)):
                    out.append(a + b)
    for cut in range(c0 + 1, c1):
        for k in range(1, max_parts):
            for a in _guillotine_partitions(r0, r1, c0, cut, k):
                for b in _guillotine_partitions(r0, r1, cut, c1, max_parts - len(a)):
                    out.append(a + b)
    return out


@pytest.mark.parametrize("seed", range(8))
def test_heuristic_is_within_a_small_factor_of_the_exhaustive_optimum(seed):
    """Not a pin of optimality (the paper's solver is unavailable), but a guard against an absurd
    plan: on instances small enough to enumerate every assignment of rectangles to devices
    (one K-slice, one rectangle per device, idle devices allowed), the heuristic's makespan stays
    within 2x of the best possible one."""
    from itertools import permutations
    from oracle.cost import task_cost
    rng = np.random.default_rng(500 + seed)
    Mg, Ng = int(rng.integers(1, 4)), int(rng.integers(1, 4))
    g = 32
    D = int(rng.integers(1, 4))
    devs = small_devices(D, 900 + seed, 1 << 24, 1 << 26)
    K = 64
    o = Opts(gran_m=g, gran_n=g, gran_k=g, kslice_max=0, ksplit=1)
    p = plan([Gemm(Mg * g, Ng * g, K)], devs, o)
    best = None
    seen = set()
    for part in _guillotine_partitions(0, Mg, 0, Ng, D):
        key = tuple(sorted(part))
        if key in seen:
            continue
        seen.add(key)
        for owners in permutations(range(D), len(part)):
            cost = max(task_cost((r1 - r0) * g, (c1 - c0) * g, K, devs[k], o.b_in, o.b_out)
                       for (r0, r1, c0, c1), k in zip(part, owners))
            best = cost if best is None else min(best, cost)
    assert best is not None and best <= p.makespan_ns[0] <= 2 * best
