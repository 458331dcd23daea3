"""Pins of the block-verification oracle: the generator's published outputs, exactness of the
identity on integer data, and the size of the residual a corrupted entry leaves."""
import numpy as np

from oracle import verify
from oracle.plan import Gemm, plan_uniform


def test_splitmix64_published_outputs():
    # first outputs of a SplitMix64 generator seeded with 0 (reference implementation's sequence)
    assert verify.splitmix64_mix(0) == 0xE220A8397B1DCDAF
    assert verify.splitmix64_mix(0x9E3779B97F4A7C15) == 0x6E789E6AA1B965F4
    assert verify.splitmix64_mix(2 * 0x9E3779B97F4A7C15 & verify.MASK) == 0x06C45D188009454F


def test_signs_are_balanced_and_distinct_per_task_and_vector():
    a, b, c = verify.signs(7, 3, 0, 4096), verify.signs(7, 3, 1, 4096), verify.signs(7, 4, 0, 4096)
    assert set(np.unique(a)) == {-1.0, 1.0}
    assert abs(a.mean()) < 0.06 and abs((a * b).mean()) < 0.06 and abs((a * c).mean()) < 0.06


def test_identity_exact_on_integers_and_residual_of_a_corrupted_entry():
    rng = np.random.default_rng(0)
    M, N, K = 24, 20, 32
    A = rng.integers(-4, 5, (M, K)).astype(np.float64)
    B = rng.integers(-4, 5, (K, N)).astype(np.float64)
    p = plan_uniform([Gemm(M, N, K)], 2, 2, 2)
    for t in p.tasks:
        P = A[t.m0:t.m1, t.k0:t.k1] @ B[t.k0:t.k1, t.n0:t.n1]
        lhs, rhs, scale = verify.task_check(t, A, B, P, seed=11)
        assert lhs == rhs and scale >= abs(rhs)
        bad = P.copy(); bad[3, 5] += 0.75                    # +-1 vectors: the residual is exactly the corruption
        lhs2, rhs2, _ = verify.task_check(t, A, B, bad, seed=11)
        assert abs(lhs2 - rhs2) == 0.75
        lost = np.zeros_like(P)                                 # a block that was never computed
        l3, r3, s3 = verify.task_check(t, A, B, lost, seed=11)
        assert l3 == 0.0 and (abs(r3) > 1e-3 * s3 or s3 == 0.0)
