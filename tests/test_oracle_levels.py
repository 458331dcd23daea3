"""Pins of the level-order oracle: the level-wise cost recursion of Section 4.1 on a hand-worked
DAG, the single-rounding bf16 conversion against bit patterns and against torch's conversion, and
the level-by-level execution against the same chain written with whole-matrix products."""
import numpy as np
import pytest

import cleave_inputs as ci
from oracle import numerics as nm
from oracle.cost import devices_from_array
from oracle.levels import execute_levels, level_costs, plan_level_costs
from oracle.plan import Gemm, Opts, plan


def test_level_cost_recursion_hand_worked():
    # level 0: GEMMs of 5, 9, 7 ms; level 1: one GEMM of 4 ms; level 2: 6 and 2 ms
    # C(0) = 9, C(1) = 9 + 4 = 13, C(2) = 13 + 6 = 19
    cost = [5, 9, 7, 4, 6, 2]
    lvl = [0, 0, 0, 1, 2, 2]
    assert level_costs(cost, lvl) == [9, 13, 19]
    # order of the list does not matter, an empty level adds nothing, one level is a plain max
    assert level_costs([6, 4, 9, 2, 5, 7], [2, 1, 0, 2, 0, 0]) == [9, 13, 19]
    assert level_costs([3, 8], [0, 2]) == [3, 3, 11]
    assert level_costs([3, 8, 5], [0, 0, 0]) == [8]
    assert level_costs([], []) == []


def test_plan_level_costs_use_the_slowest_device_of_the_slowest_gemm():
    gemms, tensors, produced = ci.two_branch_chain(256, 128, 256, 128)
    devs = devices_from_array(ci.make_devices(6, 64 * ci.MB, ci.GB, 3))
    p = plan([Gemm(g.M, g.N, g.K, g.transA, g.transB) for g in gemms], devs, Opts())
    levels = [g.level for g in gemms]
    c = plan_level_costs(p, levels)
    m = p.makespan_ns
    assert c == [max(m[0], m[1]), max(m[0], m[1]) + max(m[2], m[3]), max(m[0], m[1]) + max(m[2], m[3]) + m[4]]
    # a GEMM's cost is its most loaded device's time
    load = {}
    for t in p.tasks:
        if t.gemm == 4:
            load[t.dev] = load.get(t.dev, 0) + t.cost_ns
    assert m[4] == max(load.values())


def test_bf16_rounding_bit_patterns():
    x = np.array([1.0, 1 + 2.0 ** -8, 1 + 3 * 2.0 ** -8, 257.0, 259.0, -259.0, 0.0, -0.0, 0.5, 1e5])
    want = [0x3F80, 0x3F80, 0x3F82, 0x4380, 0x4382, 0xC382, 0x0000, 0x8000, 0x3F00, 0x47C3]
    assert [int(v) for v in nm.f64_to_bf16_bits(x)] == want       # ties go to the even neighbour
    # one rounding, not two: just above a tie an fp32 detour would first drop the 2^-30 and then tie to even
    assert int(nm.f64_to_bf16_bits(np.array([1 + 2.0 ** -8 + 2.0 ** -30]))[0]) == 0x3F81
    assert int(nm.f64_to_bf16_bits(np.array([1 + 2.0 ** -8 - 2.0 ** -30]))[0]) == 0x3F80
    # round trip of every finite positive normal bf16 value is the identity
    bits = np.arange(0x0080, 0x7F80, dtype=np.uint16)
    assert np.array_equal(nm.f64_to_bf16_bits(nm.bf16_bits_to_f64(bits)), bits)


def test_bf16_rounding_equals_torch_on_fp32_values():
    import torch
    g = torch.Generator().manual_seed(5)
    x = torch.randn(200_000, generator=g) * torch.pow(10.0, torch.randint(-6, 6, (200_000,), generator=g).float())
    want = x.to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = nm.f64_to_bf16_bits(x.numpy().astype(np.float64))       # an fp32 value is exact in fp64
    assert np.array_equal(got, want)


@pytest.mark.parametrize("integer", [True, False])
def test_level_order_execution_equals_the_chain_written_out(integer):
    gemms, tensors, produced = ci.two_branch_chain(192, 64, 128, 96)
    w = ci.Workload("chain", gemms, tensors, n_devices=5, mem_range=(64 * ci.MB, ci.GB), produced=produced)
    ts = ci.make_tensors(w, integer=integer)
    bits = {k: ci.bf16_bits(t) for k, t in ts.items()}
    devs = devices_from_array(ci.workload_devices(w))
    p = plan([Gemm(g.M, g.N, g.K, g.transA, g.transB) for g in gemms], devs, Opts(gran_m=32, gran_n=32, gran_k=64, kslice_max=64))
    assert max(p.ksplit) >= 2
    C, out_bits = execute_levels(p, gemms, bits)

    f = {k: nm.bf16_bits_to_f64(v) for k, v in bits.items()}

    def rnd(x):
        return nm.bf16_bits_to_f64(nm.f64_to_bf16_bits(x))
    Ha, Hb = f["X"] @ f["Wa"], f["X"] @ f["Wb"]
    want = [Ha, Hb, rnd(Ha) @ f["Va"], rnd(Hb) @ f["Vb"], rnd(Ha).T @ rnd(Hb)]
    for g, got, ref in zip(gemms, C, want):
        if integer:
            assert np.array_equal(got, ref), g.name
        else:
            assert np.abs(got - ref).max() <= 1e-12 * max(1.0, np.abs(ref).max()), g.name
    assert np.array_equal(out_bits["Ha"], nm.f64_to_bf16_bits(Ha)) or not integer
    # a planted mistake: feeding level 1 the unrounded level-0 output changes the result
    if not integer:
        assert np.abs(Ha @ f["Va"] - C[2]).max() > 1e-6
