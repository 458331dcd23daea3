"""Pins of the numerical oracle: brute force on tiny shapes, exactness on integer inputs, a
library matmul, the summation order, and planted mistakes that must be caught."""
import numpy as np
import pytest

import cleave_inputs as ci
from oracle import check, numerics as nm
from oracle.cost import devices_from_array
from oracle.plan import Gemm, Opts, plan, plan_uniform


def triple_loop(X, W, M, N, K, transA, transB):
    """C[i,j] = sum_k A[i,k] B[k,j] from the storage definitions, nothing vectorised."""
    C = [[0.0] * N for _ in range(M)]
    for i in range(M):
        for j in range(N):
            acc = 0.0
            for k in range(K):
                a = X[k][i] if transA else X[i][k]
                b = W[j][k] if transB else W[k][j]
                acc += float(a) * float(b)
            C[i][j] = acc
    return np.array(C)


def test_bf16_widening():
    bits = np.array([0x3F80, 0xC000, 0x3DCD, 0x0000, 0x8000, 0x7F80], dtype=np.uint16)
    v = nm.bf16_bits_to_f64(bits)
    assert v[0] == 1.0 and v[1] == -2.0 and v[2] == 0.10009765625
    assert v[3] == 0.0 and np.signbit(v[4]) and np.isinf(v[5])


@pytest.mark.parametrize("transA,transB", [(0, 0), (0, 1), (1, 0), (1, 1)])
def test_decomposed_equals_bruteforce_tiny(transA, transB):
    rng = np.random.default_rng(transA * 2 + transB)
    M, N, K = 7, 9, 11
    X = rng.integers(-4, 5, (K, M) if transA else (M, K)).astype(np.float64)
    W = rng.integers(-4, 5, (N, K) if transB else (K, N)).astype(np.float64)
    ref = triple_loop(X.tolist(), W.tolist(), M, N, K, transA, transB)
    A, B = nm.op_a(X, transA), nm.op_b(W, transB)
    devs = devices_from_array(ci.make_devices(5, 1 << 20, 1 << 22, 3))
    for p in (plan_uniform([Gemm(M, N, K, transA, transB)], 3, 2, 4),
              plan([Gemm(M, N, K, transA, transB)], devs, Opts(gran_m=2, gran_n=3, gran_k=2, kslice_max=4))):
        arena = nm.execute(p, [A], [B])
        C = nm.assemble(p, arena)[0]
        assert np.array_equal(C, ref)              # integer inputs: every sum is exact
        assert np.array_equal(nm.gemm_direct(A, B), ref)


def test_gaussian_matches_library_matmul():
    w = ci.config(2, scale=16)
    ts = ci.make_tensors(w)
    devs = devices_from_array(ci.workload_devices(w))
    gemms = [Gemm(g.M, g.N, g.K, g.transA, g.transB) for g in w.gemms]
    p = plan(gemms, devs, Opts(gran_m=32, gran_n=32, gran_k=32, kslice_max=64))
    A = [nm.op_a(nm.bf16_bits_to_f64(ci.bf16_bits(ts[g.a_key])), g.transA) for g in w.gemms]
    B = [nm.op_b(nm.bf16_bits_to_f64(ci.bf16_bits(ts[g.b_key])), g.transB) for g in w.gemms]
    arena = nm.execute(p, A, B)
    assert not np.isnan(arena[[t.part_off for t in p.tasks]]).any()
    Cs = nm.assemble(p, arena)
    assert max(p.ksplit) >= 2
    for gi, C in enumerate(Cs):
        ref = np.matmul(A[gi], B[gi])
        assert np.linalg.norm(C - ref) <= 1e-12 * np.linalg.norm(ref)
        worst, scale = check.freivalds_residual(A[gi], B[gi], C, seed=gi)
        assert worst <= 1e-10 * scale


def test_tree_sum_order_is_balanced_pairwise():
    f = np.float32
    parts = [np.array([x], dtype=f) for x in (1e8, 1.0, -1e8, 1.0)]
    assert nm.tree_sum(parts)[0] == f(0.0)              # (1e8+1) + (-1e8+1): both ones are absorbed
    assert (parts[0] + parts[1] + parts[2] + parts[3])[0] == f(1.0)   # a running sum differs
    three = [np.array([x], dtype=f) for x in (1.0, 2.0 ** -24, 2.0 ** -24)]
    assert nm.tree_sum(three)[0] == f(1.0)              # (1 + e) + (e + 0) = 1 + e -> 1 (ties to even)
    assert nm.tree_sum([np.array([-0.0], dtype=f)]).view(np.uint32)[0] == 0x80000000   # S = 1: untouched
    assert nm.tree_sum([np.array([-0.0], dtype=f)] * 3).view(np.uint32)[0] == 0          # padded with +0.0


def test_planted_mistakes_are_caught():
    rng = np.random.default_rng(0)
    A = rng.standard_normal((24, 40))
    B = rng.standard_normal((40, 16))
    C = A @ B
    ok, scale = check.freivalds_residual(A, B, C, seed=1)
    assert ok <= 1e-10 * scale
    bad = C.copy(); bad[5, 7] += 1e-3                          # single-entry corruption
    assert check.freivalds_residual(A, B, bad, seed=1)[0] > 1e-6
    assert check.freivalds_residual(A, B, A[:, :-1] @ B[:-1], seed=1)[0] > 1e-6      # dropped term
    p = plan_uniform([Gemm(24, 16, 40)], 2, 2, 2)
    arena = nm.execute(p, [A], [B])
    arena2 = arena.copy()
    t = p.tasks[3]
    arena2[t.part_off:t.part_off + t.alpha * t.beta] = 0.0   # a lost partial block
    assert not np.allclose(nm.assemble(p, arena2)[0], C)
    assert np.allclose(nm.assemble(p, arena)[0], C, rtol=1e-13, atol=1e-13)
    # a dropped task leaves NaN behind: the gap cannot go unnoticed
    assert np.isnan(nm.assemble(p, nm.execute(p, [A], [B], dropped=[3]))[0]).any()


def test_sample_entries():
    rng = np.random.default_rng(2)
    A, B = rng.standard_normal((10, 12)), rng.standard_normal((12, 9))
    rows, cols = np.array([0, 3, 9]), np.array([8, 1, 4])
    c, bound = nm.sample_entries(A, B, rows, cols)
    assert np.allclose(c, (A @ B)[rows, cols]) and np.allclose(bound, (np.abs(A) @ np.abs(B))[rows, cols])


def test_sub_gemm_from_bits_matches_sub_gemm():
    w = ci.config(2, scale=16)
    ts = ci.make_tensors(w)
    p = plan([Gemm(g.M, g.N, g.K, g.transA, g.transB) for g in w.gemms],
             devices_from_array(ci.workload_devices(w)), Opts(gran_m=32, gran_n=32, gran_k=32, kslice_max=64))
    for t in p.tasks[::7]:
        g = w.gemms[t.gemm]
        a_bits, b_bits = ci.bf16_bits(ts[g.a_key]), ci.bf16_bits(ts[g.b_key])
        full = nm.sub_gemm(t, nm.op_a(nm.bf16_bits_to_f64(a_bits), g.transA), nm.op_b(nm.bf16_bits_to_f64(b_bits), g.transB))
        assert np.array_equal(nm.sub_gemm_from_bits(t, g.transA, g.transB, a_bits, b_bits), full)
