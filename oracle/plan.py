"""Planner: one GEMM -> independent sub-GEMM tasks (test infrastructure; see oracle/__init__.py).

Section 4.1 poses the plan as an optimisation (rows of A x columns of B per device, minimise the
slowest device's max(downlink, uplink, compute), subject to exact coverage, the zero-task rule and
the memory constraint) and solves it with a commercial MILP solver that is not described as an
algorithm.  This file is a deterministic integer heuristic for the same problem, extended by a
K-split (each output block may be cut into S K-slices whose partial blocks are summed at the
parameter server; S = 1 is the paper's formulation).  Steps:

  1  granule counts; choice of S (deep contractions are cut; K is also cut when the GEMM's whole
     level has fewer output cells than there are devices) and the nominal slice depth kappa_hat
  2  capacity a_k(T): largest output area device k can finish within T under each cost term and
     the memory constraint; devices that cannot take one granule cell stay idle (zero-task rule)
  3  T* = least T with sum_k a_k(T) >= S*M*N  (work proportional to capability)
  4  active devices sorted by capacity, grouped into teams of S (one member per K-slice)
  5  column strips, teams dealt to strips in snake order, strip widths and team heights by
     largest-remainder apportionment of granules in proportion to capacity
  6  enumerate rectangles x K-slices; split any task that violates the memory constraint
  7  ids, partial-arena offsets, per-task cost, per-device load, makespan

Arithmetic is exact (Python integers); the library must reproduce every number.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from math import isqrt
from typing import List, Optional, Sequence

from .cost import Device, ceil_div, tail_aware, task_cost, task_mem, NS

T_MAX = 1 << 50

FLAG_SUPERSEDED = 1
FLAG_REISSUED = 2

# Capabilities of the implicit devices of a uniform plan (one per task): effectively unbounded
# memory, 1 TFLOP/s, 1 GB/s both ways, no latency.
UNIFORM_DEVICE = Device(1 << 48, 1_000_000, 1_000_000_000, 1_000_000_000, 0, 0)


class PlanError(Exception):
    def __init__(self, code: str, msg: str = ""):
        super().__init__(f"{code}: {msg}")
        self.code = code


@dataclass(frozen=True)
class Gemm:
    M: int
    N: int
    K: int
    transA: int = 0
    transB: int = 0
    level: int = 0      # DAG level (Section 4.1): GEMMs of one level are independent and run in parallel


@dataclass(frozen=True)
class Opts:
    gran_m: int = 128
    gran_n: int = 128
    gran_k: int = 128
    kslice_max: int = 4096
    ksplit: int = 0
    ksplit_cap: int = 8
    reissue_fanout: int = 4
    b_in: int = 2
    b_out: int = 4
    tail_alpha_milli: int = 0      # > 1000: tail-aware latencies (Appendix C), Pareto shape in thousandths; 0 = off
    tail_beta_ppm: int = 50_000     # worst fraction of outcomes the CVaR averages over, in millionths (0.05)


@dataclass
class Task:
    id: int
    gemm: int
    dev: int
    parent: int
    m0: int
    m1: int
    n0: int
    n1: int
    k0: int
    k1: int
    kslice: int
    flags: int
    part_off: int
    cost_ns: int

    @property
    def alpha(self):
        return self.m1 - self.m0

    @property
    def beta(self):
        return self.n1 - self.n0

    @property
    def kappa(self):
        return self.k1 - self.k0

    def astuple(self):
        return (self.id, self.gemm, self.dev, self.parent, self.m0, self.m1, self.n0, self.n1,
                self.k0, self.k1, self.kslice, self.flags, self.part_off, self.cost_ns)


@dataclass
class Plan:
    gemms: List[Gemm]
    devices: List[Device]
    opts: Opts
    tasks: List[Task] = field(default_factory=list)
    arena_elems: int = 0
    makespan_ns: List[int] = field(default_factory=list)   # per GEMM
    ksplit: List[int] = field(default_factory=list)        # S per GEMM
    t_star: List[int] = field(default_factory=list)        # water-fill level per GEMM
    dead: List[set] = field(default_factory=list)          # per GEMM: devices lost to churn
    n_original: int = 0


def round_up(x: int, q: int) -> int:
    return ceil_div(x, q) * q


# ---------------------------------------------------------------------------------- capacity


def r_mem(mem_bytes: int, kappa_hat: int, b_in: int, b_out: int) -> int:
    """Largest r with 2*r*kappa*b_in + r*r*b_out <= mem  (square block under Eq. memory-constraint)."""
    lo, hi = 0, 1 << 32
    while lo < hi:
        mid = (lo + hi + 1) // 2
        if 2 * mid * kappa_hat * b_in + mid * mid * b_out <= mem_bytes:
            lo = mid
        else:
            hi = mid - 1
    return lo


def capacity(dev: Device, T: int, kappa_hat: int, o: Opts, rm: Optional[int] = None) -> int:
    """a_k(T): output area device k can complete within T ns for slices of depth kappa_hat."""
    if T <= dev.dl_lat_ns:
        a_dl = 0
    else:
        s = ((T - dev.dl_lat_ns) * dev.dl_Bps) // (NS * kappa_hat * o.b_in)   # alpha + beta affordable
        a_dl = (s // 2) * (s - s // 2)                                        # square maximises area
    if T <= dev.ul_lat_ns:
        a_ul = 0
    else:
        a_ul = ((T - dev.ul_lat_ns) * dev.ul_Bps) // (NS * o.b_out)
    a_comp = (T * dev.flops_mflops) // (2000 * kappa_hat)
    if rm is None:
        rm = r_mem(dev.mem_bytes, kappa_hat, o.b_in, o.b_out)
    a = min(a_dl, a_ul, a_comp, rm * rm)
    if a < o.gran_m * o.gran_n:          # zero-task rule: cannot take a single cell -> idle
        return 0
    return a


def apportion(total: int, weights: Sequence[int]) -> List[int]:
    """Split `total` units over len(weights) parts, each >= 1, the rest in proportion to the
    weights by largest remainder (ties to the lower index)."""
    n = len(weights)
    assert total >= n >= 1
    W = sum(weights)
    rest = total - n
    q = [(rest * w) // W for w in weights]
    rem = [rest * w - qi * W for w, qi in zip(weights, q)]
    left = rest - sum(q)
    order = sorted(range(n), key=lambda i: (-rem[i], i))
    for i in order[:left]:
        q[i] += 1
    return [1 + qi for qi in q]


def split_counts(total: int, parts: int) -> List[int]:
    """`total` units in `parts` consecutive parts: floor(total/parts), the first total%parts get +1."""
    return [total // parts + (1 if i < total % parts else 0) for i in range(parts)]


# ---------------------------------------------------------------------------------- one GEMM


def choose_ksplit(g: Gemm, n_dev: int, o: Opts, level_cells: int, Kg: int) -> int:
    """`level_cells`: output cells of all GEMMs of this GEMM's level together.  The GEMMs of a level
    run in parallel over the same devices (Section 4.1), so devices are only left without a cell,
    and K is only split to give them work, when the whole level has fewer cells than devices."""
    if o.ksplit:
        return max(1, min(o.ksplit, Kg))
    s_depth = ceil_div(g.K, o.kslice_max) if o.kslice_max else 1
    s_fan = ceil_div(n_dev, level_cells)
    return max(1, min(max(s_depth, s_fan), o.ksplit_cap, Kg))


def output_cells(g: Gemm, o: Opts) -> int:
    return ceil_div(g.M, o.gran_m) * ceil_div(g.N, o.gran_n)


def plan_rectangles(g: Gemm, devices: Sequence[Device], o: Opts, level_cells: Optional[int] = None):
    """Steps 1-6 for one GEMM.  Returns (S, T*, [(m0,m1,n0,n1,k0,k1,kslice,dev), ...]).
    `level_cells` defaults to the GEMM's own cells (a level of its own)."""
    if g.M <= 0 or g.N <= 0 or g.K <= 0:
        raise PlanError("E_INVAL", "empty GEMM")
    if not devices:
        raise PlanError("E_NO_DEVICES")
    Mg, Ng, Kg = ceil_div(g.M, o.gran_m), ceil_div(g.N, o.gran_n), ceil_div(g.K, o.gran_k)
    S = choose_ksplit(g, len(devices), o, Mg * Ng if level_cells is None else level_cells, Kg)
    s_limit = S if o.ksplit else min(o.ksplit_cap, Kg)

    while True:
        kappa_hat = min(g.K, o.gran_k * ceil_div(Kg, S))
        rms = [r_mem(d.mem_bytes, kappa_hat, o.b_in, o.b_out) for d in devices]
        need = S * g.M * g.N

        def total(T):
            return sum(capacity(d, T, kappa_hat, o, rm) for d, rm in zip(devices, rms))

        if total(T_MAX) >= need:
            lo, hi = 0, T_MAX
            while lo < hi:
                mid = (lo + hi) // 2
                if total(mid) >= need:
                    hi = mid
                else:
                    lo = mid + 1
            t_star = lo
            break
        if S + 1 > s_limit:
            raise PlanError("E_INFEASIBLE", "devices cannot hold the GEMM at any makespan")
        S += 1

    caps = [capacity(d, t_star, kappa_hat, o, rm) for d, rm in zip(devices, rms)]
    active = sorted((k for k in range(len(devices)) if caps[k] > 0), key=lambda k: (-caps[k], k))
    n_act = len(active)
    n_teams = max(1, min(n_act // S, Mg * Ng))
    teams = [[active[(j * S + s) % n_act] for s in range(S)] for j in range(n_teams)]
    weights = [sum(caps[k] for k in team) for team in teams]

    c = max(1, min(isqrt((n_teams * Ng) // Mg), n_teams, Ng))
    while ceil_div(n_teams, c) > Mg:
        c += 1
    strips: List[List[int]] = [[] for _ in range(c)]
    for j in range(n_teams):
        r = j % (2 * c)
        strips[r if r < c else 2 * c - 1 - r].append(j)
    for members in strips:
        if not members or len(members) > Mg:
            raise PlanError("E_INFEASIBLE", "strip deal failed")
    widths = apportion(Ng, [sum(weights[j] for j in members) for members in strips])
    kparts = split_counts(Kg, S)

    rects = []
    col_g = 0
    for members, wg in zip(strips, widths):
        n0, n1 = col_g * o.gran_n, min(g.N, (col_g + wg) * o.gran_n)
        heights = apportion(Mg, [weights[j] for j in members])
        row_g = 0
        for j, hg in zip(members, heights):
            m0, m1 = row_g * o.gran_m, min(g.M, (row_g + hg) * o.gran_m)
            kg = 0
            for s in range(S):
                k0, k1 = kg * o.gran_k, min(g.K, (kg + kparts[s]) * o.gran_k)
                dev = teams[j][s]
                rects.extend(_memory_repair(m0, m1, n0, n1, k0, k1, s, dev, devices[dev], o))
                kg += kparts[s]
            row_g += hg
        col_g += wg
    return S, t_star, rects


def _memory_repair(m0, m1, n0, n1, k0, k1, s, dev, d: Device, o: Opts):
    """Depth-first split of a task that violates Eq. (memory-constraint); pieces stay on `dev`."""
    if task_mem(m1 - m0, n1 - n0, k1 - k0, o.b_in, o.b_out) <= d.mem_bytes:
        return [(m0, m1, n0, n1, k0, k1, s, dev)]
    rg, cg = ceil_div(m1 - m0, o.gran_m), ceil_div(n1 - n0, o.gran_n)
    if rg >= cg and rg > 1:
        mid = m0 + ceil_div(rg, 2) * o.gran_m
        return (_memory_repair(m0, mid, n0, n1, k0, k1, s, dev, d, o) +
                _memory_repair(mid, m1, n0, n1, k0, k1, s, dev, d, o))
    if cg > 1:
        mid = n0 + ceil_div(cg, 2) * o.gran_n
        return (_memory_repair(m0, m1, n0, mid, k0, k1, s, dev, d, o) +
                _memory_repair(m0, m1, mid, n1, k0, k1, s, dev, d, o))
    raise PlanError("E_INFEASIBLE", "one granule cell exceeds device memory")


# ---------------------------------------------------------------------------------- whole plans


def _finish(plan: Plan, per_gemm_rects):
    """Step 7: ids (GEMM-major, enumeration order), arena offsets, costs, loads, makespans."""
    o = plan.opts
    off = 0
    for gi, rects in enumerate(per_gemm_rects):
        load = {}
        for (m0, m1, n0, n1, k0, k1, s, dev) in rects:
            tid = len(plan.tasks)
            cost = task_cost(m1 - m0, n1 - n0, k1 - k0, plan.devices[dev], o.b_in, o.b_out)
            plan.tasks.append(Task(tid, gi, dev, tid, m0, m1, n0, n1, k0, k1, s, 0, off, cost))
            off += round_up((m1 - m0) * (n1 - n0), 32)
            load[dev] = load.get(dev, 0) + cost
        plan.makespan_ns.append(max(load.values()))
        plan.dead.append(set())
    plan.arena_elems = off
    plan.n_original = len(plan.tasks)
    return plan


def plan(gemms: Sequence[Gemm], devices: Sequence[Device], opts: Opts = Opts()) -> Plan:
    """Every GEMM is planned independently over the same device list (each GEMM is its own
    dispatch round; a schedule is computed when the device set changes and kept until it changes
    again, Section 3.2)."""
    if opts.tail_alpha_milli:
        # tail-aware cost (Appendix C, Eq. 23): every latency overhead enters with its CVaR (Eq. 24)
        devices = [tail_aware(d, opts.tail_alpha_milli, opts.tail_beta_ppm) for d in devices]
    p = Plan(list(gemms), list(devices), opts)
    per_gemm = []
    cells = {}
    for g in gemms:
        if g.M > 0 and g.N > 0:
            cells[g.level] = cells.get(g.level, 0) + output_cells(g, opts)
    for g in gemms:
        S, t_star, rects = plan_rectangles(g, devices, opts, cells.get(g.level))
        p.ksplit.append(S)
        p.t_star.append(t_star)
        per_gemm.append(rects)
    return _finish(p, per_gemm)


def plan_uniform(gemms: Sequence[Gemm], grid_m: int, grid_n: int, ksplit: int,
                 opts: Opts = Opts()) -> Plan:
    """Uniform grid: rows in grid_m parts, columns in grid_n parts, K in ksplit parts (sizes
    floor + 1 for the first remainder parts); ids block-row-major then slice; one implicit
    device per task (device index restarts at 0 for every GEMM)."""
    n_per = grid_m * grid_n * ksplit
    p = Plan(list(gemms), [UNIFORM_DEVICE] * n_per, opts)
    per_gemm = []
    for g in gemms:
        if grid_m < 1 or grid_n < 1 or ksplit < 1 or grid_m > g.M or grid_n > g.N or ksplit > g.K:
            raise PlanError("E_INVAL", "grid larger than the GEMM")
        rects = []
        hm, wn, dk = split_counts(g.M, grid_m), split_counts(g.N, grid_n), split_counts(g.K, ksplit)
        m0 = 0
        for i in range(grid_m):
            n0 = 0
            for j in range(grid_n):
                k0 = 0
                for s in range(ksplit):
                    rects.append((m0, m0 + hm[i], n0, n0 + wn[j], k0, k0 + dk[s], s, len(rects)))
                    k0 += dk[s]
                n0 += wn[j]
            m0 += hm[i]
        p.ksplit.append(ksplit)
        p.t_star.append(0)
        per_gemm.append(rects)
    return _finish(p, per_gemm)
