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
    # 16 identical devices, Mg = Ng = 8, S = 1 -> 4 x 4 grid of equal 256 x 256 blocks
    devs = devices_from_array(ci.homogeneous_devices(16))
    p = plan([Gemm(1024, 1024, 512)], devs, Opts(kslice_max=0))
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
    assert plan([Gemm(256, 256, 8192)], devs[:4], Opts()).ksplit == [2]        # depth cap 4096
    assert plan([Gemm(256, 256, 11008)], devs[:4], Opts()).ksplit == [3]
    assert plan([Gemm(256, 256, 4096)], devs[:4], Opts()).ksplit == [1]
    assert plan([Gemm(256, 256, 4096)], devs[:4], Opts(kslice_max=2048)).ksplit == [2]
    # more devices than output cells -> split K so that all can work (2x2 cells, 8 devices)
    assert plan([Gemm(256, 256, 512)], devs, Opts()).ksplit == [2]
    # ... unless the GEMM's level holds enough cells for every device: four such GEMMs in one level are 16
    # cells for 8 devices (no split), the same four in four levels are split as before
    four = [Gemm(256, 256, 512, level=0)] * 4
    assert plan(four, devs, Opts()).ksplit == [1, 1, 1, 1]
    assert plan([Gemm(256, 256, 512, level=i) for i in range(4)], devs, Opts()).ksplit == [2, 2, 2, 2]
    assert plan([Gemm(256, 256, 512, level=0), Gemm(256, 256, 512, level=0), Gemm(256, 256, 512, level=1)], devs,
                Opts()).ksplit == [1, 1, 2]
    # K-slices are consecutive, granule aligned, sizes differ by at most one granule
    p = plan([Gemm(256, 256, 11008)], devs[:4], Opts())
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


# ---------------------------------------------------------------------------------- capacity and T*
# The water-fill capacity a_k(T) is a closed form that follows from the cost terms of Section 4.1
# (pinned in test_oracle_cost.py on the paper's worked example) and the memory constraint.  It is
# pinned here three ways: hand-computed areas on devices where exactly one term binds, agreement
# with a brute-force search that only calls the cost functions, and the defining property of each
# term (the returned area is affordable within T, the next larger one is not).

from oracle.cost import c_comp, c_dl, c_ul

BIG = 10 ** 15
CAP_OPTS = Opts(gran_m=1, gran_n=1, gran_k=1)


def _one_binding_term_devices():
    """(device, T, kappa_hat, hand-computed area, name of the binding term)"""
    return [
        # downlink: (T - L^d) W^d / (1e9 * kappa * b_in) = 2e6 * 1e6 / (1e9 * 200) = 10 rows + columns -> 5 x 5
        (Device(BIG, BIG, 10 ** 6, BIG, 1000, 0), 1000 + 2 * 10 ** 6, 100, 25, "dl"),
        # an odd budget of rows + columns: 11 -> 5 x 6
        (Device(BIG, BIG, 10 ** 6, BIG, 1000, 0), 1000 + 22 * 10 ** 5, 100, 30, "dl"),
        # uplink: (T - L^u) W^u / (1e9 * b_out) = 1e5 * 1e6 / 4e9 = 25 outputs
        (Device(BIG, BIG, BIG, 10 ** 6, 0, 500), 500 + 10 ** 5, 100, 25, "ul"),
        # compute: T F / (2000 kappa) = 1e5 * 1000 / 2e5 = 500 outputs  (F = 1000 MFLOP/s)
        (Device(BIG, 1000, BIG, BIG, 0, 0), 10 ** 5, 100, 500, "comp"),
        # memory: 2 r kappa b_in + r^2 b_out <= 4500 -> r = 10 (4400), r = 11 needs 4884
        (Device(4500, BIG, BIG, BIG, 0, 0), 10 ** 5, 100, 100, "mem"),
    ]


@pytest.mark.parametrize("case", range(5))
def test_capacity_hand_computed_one_binding_term(case):
    dev, T, kappa, want, which = _one_binding_term_devices()[case]
    assert capacity(dev, T, kappa, CAP_OPTS) == want
    # the latency is paid before the first byte: at T = L nothing can be done yet
    if which == "dl":
        assert capacity(dev, dev.dl_lat_ns, kappa, CAP_OPTS) == 0
        # long before the latency has passed the (negative) time left must not turn into an area
        late = dev._replace(dl_lat_ns=10 ** 7)
        assert capacity(late, 10, kappa, CAP_OPTS) == 0 and capacity(late, 10 ** 7 - 1, kappa, CAP_OPTS) == 0
        assert capacity(dev, T - 1, kappa, CAP_OPTS) < want          # T is the first instant the area fits
    if which == "ul":
        assert capacity(dev, dev.ul_lat_ns, kappa, CAP_OPTS) == 0
        assert capacity(dev, T - 1, kappa, CAP_OPTS) == want - 1
    if which == "comp":
        # depth matters: twice the slice depth halves the affordable area
        assert capacity(dev, T, 2 * kappa, CAP_OPTS) == want // 2
    if which == "mem":
        assert capacity(dev, 10 * T, kappa, CAP_OPTS) == want          # time does not help


def _capacity_bruteforce(dev, T, kappa, o, limit=40):
    """min over the four terms of the largest area that term alone allows, found by trying blocks
    with the cost functions themselves: every (alpha, beta) up to `limit` for the downlink (its cost
    depends on alpha + beta), every 1 x n block for uplink and compute (their cost depends on the
    area only), every square for the memory constraint."""
    best = {"dl": 0, "ul": 0, "comp": 0}
    for a in range(1, limit + 1):
        for b in range(1, limit + 1):
            if c_dl(a, b, kappa, dev, o.b_in) <= T:
                best["dl"] = max(best["dl"], a * b)
    for n in range(1, limit * limit + 1):
        if c_ul(1, n, dev, o.b_out) <= T:
            best["ul"] = n
        if c_comp(1, n, kappa, dev) <= T:
            best["comp"] = n
    r = 0
    while task_mem(r + 1, r + 1, kappa, o.b_in, o.b_out) <= dev.mem_bytes:
        r += 1
    area = min(best["dl"], best["ul"], best["comp"], r * r)
    return area if area >= o.gran_m * o.gran_n else 0


def test_capacity_equals_bruteforce_over_the_cost_functions():
    stats = {"compared": 0, "working": 0}
    for seed in range(10):
        _compare_capacity_with_bruteforce(np.random.default_rng(40 + seed), stats)
    assert stats["compared"] >= 200 and stats["working"] >= 50     # idle and working instants both occur


def _compare_capacity_with_bruteforce(rng, stats):
    kappa = int(rng.integers(1, 64))
    # rates chosen so that the affordable block stays well inside the brute-force search window
    dev = Device(int(rng.integers(2_000, 40_000)), int(rng.integers(50, 2_000)), int(rng.integers(10 ** 5, 10 ** 7)),
                 int(rng.integers(10 ** 5, 10 ** 7)), int(rng.integers(0, 3_000)), int(rng.integers(0, 3_000)))
    o = Opts(gran_m=int(rng.integers(1, 4)), gran_n=int(rng.integers(1, 4)), gran_k=1)
    # instants from 0 up to where a cost term reaches the edge of the brute-force search window
    limit = 40

    def clipped(T):
        return (c_dl(limit, limit + 1, kappa, dev, o.b_in) <= T or c_ul(1, limit * limit, dev, o.b_out) <= T or
                c_comp(1, limit * limit, kappa, dev) <= T)
    t_hi = 1
    while not clipped(2 * t_hi):
        t_hi *= 2
    for T in [int(x) for x in rng.integers(0, t_hi, 40)] + [dev.dl_lat_ns, dev.ul_lat_ns, dev.dl_lat_ns + 1]:
        if clipped(T):
            continue
        got = capacity(dev, T, kappa, o)
        assert got == _capacity_bruteforce(dev, T, kappa, o, limit), (T, kappa, dev)
        stats["compared"] += 1
        stats["working"] += got > 0


def test_capacity_defining_property_at_config_scale():
    """On the synthetic devices of the Llama-7B-shaped workload: the square block of the returned
    area is affordable within T under every cost term, and for the term that binds, one more
    row + column (downlink) or one more output (uplink, compute) is not."""
    w = ci.config(3)
    devs = devices_from_array(ci.workload_devices(w))[:64]
    o = Opts(gran_m=128, gran_n=128, gran_k=128)
    kappa = 4096
    for T in (30_000_000, 400_000_000, 3_000_000_000):
        for d in devs:
            a = capacity(d, T, kappa, o)
            if a == 0:
                continue
            side = isqrt_(a)
            assert c_dl(side, side, kappa, d, o.b_in) <= T
            assert c_ul(side, side, d, o.b_out) <= T and c_ul(1, a, d, o.b_out) <= T
            assert c_comp(side, side, kappa, d) <= T and c_comp(1, a, kappa, d) <= T
            assert task_mem(side, side, kappa, o.b_in, o.b_out) <= d.mem_bytes
            # which term binds: the one whose own maximum equals the returned area
            s = 0 if T <= d.dl_lat_ns else ((T - d.dl_lat_ns) * d.dl_Bps) // (10 ** 9 * kappa * o.b_in)
            binding = []
            if (s // 2) * (s - s // 2) == a:
                binding.append("dl")
                assert c_dl(s // 2, s - s // 2, kappa, d, o.b_in) <= T < c_dl(s // 2, s - s // 2 + 1, kappa, d, o.b_in)
            if c_ul(1, a + 1, d, o.b_out) > T:
                binding.append("ul")
            if c_comp(1, a + 1, kappa, d) > T:
                binding.append("comp")
            r = r_mem(d.mem_bytes, kappa, o.b_in, o.b_out)
            if r * r == a:
                binding.append("mem")
                assert task_mem(r + 1, r + 1, kappa, o.b_in, o.b_out) > d.mem_bytes
            assert binding, (d, T, a)


def isqrt_(x):
    from math import isqrt
    return isqrt(x)


def test_t_star_two_devices_by_hand():
    """Water-fill level of a 20 x 20 x 100 GEMM (one slice, 400 outputs) on two compute-bound
    devices of 1000 and 3000 MFLOP/s: a_k(T) = floor(T F_k / 2e5), so 400 outputs need
    T (1000 + 3000) / 2e5 >= 400 up to the two floors: T = 20000 ns gives 100 + 300 exactly and
    T = 19999 gives 99 + 299."""
    devs = [Device(BIG, 1000, BIG, BIG, 0, 0), Device(BIG, 3000, BIG, BIG, 0, 0)]
    o = Opts(gran_m=1, gran_n=1, gran_k=1, kslice_max=0, ksplit=1)
    p = plan([Gemm(20, 20, 100)], devs, o)
    assert p.t_star == [20000]
    assert capacity(devs[0], 20000, 100, o) + capacity(devs[1], 20000, 100, o) == 400
    assert capacity(devs[0], 19999, 100, o) + capacity(devs[1], 19999, 100, o) == 398
    # with a downlink latency of 7000 ns on the fast device and a link that makes the downlink bind:
    # s = floor((T - 7000) * 1e9 / (1e9 * 200)) rows + columns on device 1, compute bound on device 0
    devs2 = [Device(BIG, 1000, BIG, BIG, 0, 0), Device(BIG, BIG, 10 ** 9, BIG, 7000, 0)]
    p2 = plan([Gemm(20, 20, 100)], devs2, o)
    T = p2.t_star[0]

    def total(t):
        s = 0 if t <= 7000 else (t - 7000) // 200
        return (t * 1000) // 200000 + (s // 2) * (s - s // 2)
    assert total(T) >= 400 > total(T - 1)
    # at 14400: s = 37 -> 18 * 19 = 342, plus floor(14400 / 200) = 72 -> 414; at 14399: s = 36 -> 324 + 71 = 395
    assert T == 14400


@pytest.mark.parametrize("seed", range(6))
def test_t_star_is_the_least_feasible_level_by_linear_scan(seed):
    rng = np.random.default_rng(70 + seed)
    D = int(rng.integers(1, 5))
    devs = [Device(int(rng.integers(20_000, 200_000)), int(rng.integers(200, 2_000)), int(rng.integers(10 ** 6, 10 ** 7)),
                   int(rng.integers(10 ** 6, 10 ** 7)), int(rng.integers(0, 2_000)), int(rng.integers(0, 2_000)))
            for _ in range(D)]
    o = Opts(gran_m=2, gran_n=2, gran_k=4, kslice_max=0, ksplit=1)
    g = Gemm(int(rng.integers(4, 14)), int(rng.integers(4, 14)), int(rng.integers(4, 32)))
    try:
        p = plan([g], devs, o)
    except PlanError:
        pytest.skip("infeasible draw")
    kappa = min(g.K, o.gran_k * -(-g.K // o.gran_k))
    need = g.M * g.N
    T = p.t_star[0]
    assert sum(capacity(d, T, kappa, o) for d in devs) >= need
    # no earlier instant suffices: the capacities (pinned above) never decrease with T, checked here on
    # a scan of the instants below T* together with the sum itself
    step = max(1, T // 3000)
    prev = 0
    for t in list(range(0, T, step)) + [T - 1]:
        tot = sum(capacity(d, t, kappa, o) for d in devs)
        assert tot < need
        if t < T - 1 or t % step == 0:
            assert tot >= prev
            prev = tot
