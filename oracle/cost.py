"""Cost model of Section 4.1 (test infrastructure; see oracle/__init__.py).

All quantities are Python integers: times in nanoseconds, sizes in bytes, bandwidths in bytes/s,
compute rate F in MFLOP/s.  Divisions round up, so a cost is never under-estimated.

A task is an (alpha x beta) output block over a K-range of length kappa.  With kappa = n_s (one
K-slice) these are exactly the paper's per-device terms.
"""
from __future__ import annotations

from typing import NamedTuple

NS = 10 ** 9


class Device(NamedTuple):
    """Device record of Section 4.1: M_k, F_k, W^d_k, W^u_k, L^d_k, L^u_k."""
    mem_bytes: int
    flops_mflops: int
    dl_Bps: int
    ul_Bps: int
    dl_lat_ns: int
    ul_lat_ns: int


def devices_from_array(arr):
    return [Device(*(int(x) for x in row)) for row in arr]


def ceil_div(a: int, b: int) -> int:
    return -((-a) // b)


def c_dl(alpha: int, beta: int, kappa: int, dev: Device, b_in: int, latency: bool = True) -> int:
    """Downlink term, Eq. (ul-dl-cost): (alpha*n*b + n*beta*b) / W^d + L^d.

    `latency=False` gives the churn-recovery form of Section 4.2, which has no L^d term."""
    t = ceil_div((alpha + beta) * kappa * b_in * NS, dev.dl_Bps)
    return t + (dev.dl_lat_ns if latency else 0)


def c_ul(alpha: int, beta: int, dev: Device, b_out: int) -> int:
    """Uplink term, Eq. (ul-dl-cost): alpha*beta*b / W^u + L^u."""
    return ceil_div(alpha * beta * b_out * NS, dev.ul_Bps) + dev.ul_lat_ns


def c_comp(alpha: int, beta: int, kappa: int, dev: Device) -> int:
    """Computation term, Eq. (computation-cost): 2*alpha*beta*n / F  (F in MFLOP/s -> ns)."""
    return ceil_div(2 * alpha * beta * kappa * 1000, dev.flops_mflops)


def task_cost(alpha, beta, kappa, dev: Device, b_in: int, b_out: int) -> int:
    """Eq. (communication-cost): downlink, uplink and compute overlap -> max of the three."""
    return max(c_dl(alpha, beta, kappa, dev, b_in), c_ul(alpha, beta, dev, b_out),
               c_comp(alpha, beta, kappa, dev))


def task_mem(alpha, beta, kappa, b_in: int, b_out: int) -> int:
    """Left side of Eq. (memory-constraint): rows + columns + output block resident together."""
    return (alpha + beta) * kappa * b_in + alpha * beta * b_out


def lower_bound_ns(gemm_flops: int, devices) -> int:
    """Eq. 18 for one GEMM in a level: max(total work / total rate, work / fastest rate) is a
    bound for the *indivisible* unit; with row-column divisible work only the first term binds a
    single GEMM.  Returned: floor(W / sum F) in ns (a lower bound on any plan's makespan)."""
    total_f = sum(d.flops_mflops for d in devices)
    return (gemm_flops * 1000) // total_f


def tail_latency_scale_q20(alpha_milli: int, beta_ppm: int) -> int:
    """Tail-aware latency (Appendix C, Eqs. 20, 23, 24): a latency overhead is modelled as Pareto
    with shape alpha and scale x_m = the device's stated overhead, and enters the cost with its
    conditional value-at-risk over the worst beta-fraction of outcomes,
        CVaR_beta[L] = x_m / beta^(1/alpha) * alpha / (alpha - 1)          (alpha > 1).
    Returned: floor(2^20 * CVaR_beta[L] / x_m), from alpha in thousandths and beta in millionths.
    (One floating-point power; the integer result is what plans are built from.)"""
    if alpha_milli <= 1000 or not (0 < beta_ppm <= 1_000_000):
        raise ValueError("tail model needs alpha > 1 and 0 < beta <= 1")
    import math
    a = alpha_milli / 1000.0
    b = beta_ppm / 1000000.0
    f = (a / (a - 1.0)) * math.pow(b, -1.0 / a)
    return int(math.floor(f * 1048576.0))


def tail_aware(dev: Device, alpha_milli: int, beta_ppm: int) -> Device:
    """The device with both latency overheads replaced by their CVaR (rounded up to whole ns)."""
    q = tail_latency_scale_q20(alpha_milli, beta_ppm)
    return dev._replace(dl_lat_ns=ceil_div(dev.dl_lat_ns * q, 1 << 20), ul_lat_ns=ceil_div(dev.ul_lat_ns * q, 1 << 20))
