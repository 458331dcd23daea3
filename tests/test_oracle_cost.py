"""Pins of the cost evaluator: the worked example the paper prints (Section 5.2)."""
import pytest
from conftest import read_golden
from oracle.cost import Device, c_comp, c_dl, c_ul, task_cost, task_mem, ceil_div

G = read_golden("worked_example_512dev_llama2_13b.txt")

# The printed numbers are reproduced by a shard of alpha = m / D = 256 rows and beta = q / D
# columns with latency overheads 5 ms down / 10 ms up (the paper never states the overheads; its
# alpha = beta = 10 does not give its own numbers).
MEDIAN = Device(8 << 30, int(G["flops"] / 1e6), int(G["dl_Bps"]), int(G["ul_Bps"]), 5_000_000, 10_000_000)
ALPHA = 128 * 1024 // int(G["devices"])


def test_level_costs_match_paper():
    h = int(G["h"])
    beta = h // int(G["devices"])
    assert ALPHA == 256 and beta == 10
    assert abs(c_dl(ALPHA, beta, h, MEDIAN, 2) / 1e9 - G["c_dl_s"]) < 0.5e-4
    assert abs(c_ul(ALPHA, beta, MEDIAN, 2) / 1e9 - G["c_ul_s"]) < 0.5e-4
    assert abs(c_comp(ALPHA, beta, h, MEDIAN) / 1e9 - G["c_comp_s"]) < 0.5e-7
    # level is downlink dominated
    assert task_cost(ALPHA, beta, h, MEDIAN, 2, 2) == c_dl(ALPHA, beta, h, MEDIAN, 2)


def test_per_batch_time_matches_paper():
    h, H, D = int(G["h"]), int(G["H"]), int(G["devices"])
    per_layer = (4 * task_cost(ALPHA, h // D, h, MEDIAN, 2, 2)      # four h x h GEMMs
                 + task_cost(ALPHA, H // D, h, MEDIAN, 2, 2)        # one h x H GEMM
                 + task_cost(ALPHA, h // D, H, MEDIAN, 2, 2))       # one H x h GEMM
    total_s = per_layer * int(G["layers"]) / 1e9
    assert abs(total_s - G["per_batch_s"]) < 0.05


def test_closed_forms():
    d = Device(10 ** 9, 1_000_000, 1_000_000, 500_000, 7, 11)
    # (alpha + beta) * kappa * b bytes at 1 MB/s -> microseconds * 1000 ns, plus latency
    assert c_dl(3, 5, 10, d, 2) == (3 + 5) * 10 * 2 * 1000 + 7
    assert c_dl(3, 5, 10, d, 2, latency=False) == (3 + 5) * 10 * 2 * 1000
    assert c_ul(3, 5, d, 4) == 3 * 5 * 4 * 2000 + 11
    assert c_comp(3, 5, 10, d) == ceil_div(2 * 3 * 5 * 10 * 1000, 1_000_000) == 1
    # symmetric in alpha <-> beta; monotone in every argument
    assert task_cost(3, 5, 10, d, 2, 4) == task_cost(5, 3, 10, d, 2, 4)
    assert task_cost(4, 5, 10, d, 2, 4) >= task_cost(3, 5, 10, d, 2, 4)
    assert task_mem(3, 5, 10, 2, 4) == 3 * 10 * 2 + 10 * 5 * 2 + 3 * 5 * 4


# ---- tail-aware latency (Appendix C): CVaR of a Pareto-distributed overhead, Eq. 24

def test_tail_latency_scale_closed_forms():
    from oracle.cost import tail_latency_scale_q20
    one = 1 << 20
    # beta = 1: the CVaR over all outcomes is the mean of the Pareto law, x_m * alpha / (alpha - 1)
    assert tail_latency_scale_q20(2000, 1_000_000) == 2 * one
    assert tail_latency_scale_q20(5000, 1_000_000) == (5 * one) // 4
    # alpha = 4, beta = 1/16: beta^(1/4) = 1/2, factor (4/3) / (1/2) = 8/3
    assert tail_latency_scale_q20(4000, 62_500) == (8 * one) // 3
    # alpha = 2: factor^2 = 4 / beta exactly; beta = 0.05 (the paper's recommended 95th-percentile setting) -> 80
    q = tail_latency_scale_q20(2000, 50_000)
    assert q * q <= 80 * one * one < (q + 1) * (q + 1)
    # heavier tails and rarer outcomes cost more
    assert tail_latency_scale_q20(1500, 50_000) > tail_latency_scale_q20(2000, 50_000) > tail_latency_scale_q20(3000, 50_000)
    assert tail_latency_scale_q20(2000, 10_000) > tail_latency_scale_q20(2000, 50_000)
    for bad in ((1000, 50_000), (900, 50_000), (2000, 0), (2000, 1_000_001)):
        with pytest.raises(ValueError):
            tail_latency_scale_q20(*bad)


def test_tail_latency_scale_against_sampled_pareto():
    """Independent of the closed form: draw Pareto latencies by inverse transform (Eq. 20:
    P(L > x) = (x_m / x)^alpha) and average the worst beta-fraction."""
    import numpy as np
    from oracle.cost import tail_latency_scale_q20
    rng = np.random.default_rng(11)
    for alpha, beta in ((3.0, 0.05), (4.0, 0.10), (2.5, 0.25)):
        x = rng.random(4_000_000) ** (-1.0 / alpha)          # x_m = 1
        x.sort()
        worst = x[int(round((1 - beta) * len(x))):].mean()
        f = tail_latency_scale_q20(int(alpha * 1000), int(beta * 1_000_000)) / (1 << 20)
        assert abs(worst - f) <= 0.03 * f, (alpha, beta, worst, f)


def test_tail_aware_device_and_plan():
    from oracle.cost import Device, tail_aware, tail_latency_scale_q20
    from oracle.plan import Gemm, Opts, plan
    d = Device(1 << 30, 6_000_000, 55_000_000, 7_500_000, 5_000_000, 10_000_001)
    # factor 8/3 held with 20 fractional bits (2796202 / 2^20 = 2.66666603...), products rounded up to whole ns:
    # 5,000,000 * 2796202 / 1048576 = 13,333,330.2 -> 13,333,331; 10,000,001 * 2796202 / 1048576 = 26,666,663.0 -> 26,666,663
    t = tail_aware(d, 4000, 62_500)
    assert (t.dl_lat_ns, t.ul_lat_ns) == (13_333_331, 26_666_663)
    assert t[:4] == d[:4]
    # a plan under the tail-aware cost is the plan of the devices with CVaR latencies, and it is slower on paper
    devs = [d._replace(dl_Bps=55_000_000 + 1000 * i, flops_mflops=6_000_000 + 10_000 * i) for i in range(12)]
    g = [Gemm(1024, 768, 512)]
    plain = plan(g, devs, Opts())
    tail = plan(g, devs, Opts(tail_alpha_milli=4000, tail_beta_ppm=62_500))
    by_hand = plan(g, [tail_aware(x, 4000, 62_500) for x in devs], Opts())
    assert [x.astuple() for x in tail.tasks] == [x.astuple() for x in by_hand.tasks]
    assert tail.t_star[0] > plain.t_star[0] and tail.makespan_ns[0] > plain.makespan_ns[0]
    q = tail_latency_scale_q20(4000, 62_500)
    assert tail.devices[3].ul_lat_ns == -((-devs[3].ul_lat_ns * q) // (1 << 20))
