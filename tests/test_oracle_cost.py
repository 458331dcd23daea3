"""Pins of the cost evaluator: the worked example the paper prints (Section 5.2)."""
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
