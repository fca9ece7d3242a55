"""Pins for the GEMM oracle (CPU only)."""
import numpy as np

from oracle import gemm as G


def test_triple_loop_on_tiny_inputs():
    rng = np.random.default_rng(0)
    a = rng.standard_normal((5, 7)); b = rng.standard_normal((4, 7))
    ref = [[sum(float(a[i, k]) * float(b[j, k]) for k in range(7)) for j in range(4)] for i in range(5)]
    assert np.max(np.abs(G.gemm_nt(a, b) - np.array(ref))) < 1e-13


def test_exact_on_small_integers():
    rng = np.random.default_rng(1)
    a = rng.integers(-9, 10, (6, 11)); b = rng.integers(-9, 10, (8, 11))
    exact = np.array([[int(sum(int(a[i, k]) * int(b[j, k]) for k in range(11))) for j in range(8)] for i in range(6)])
    assert np.array_equal(G.gemm_nt(a, b), exact.astype(np.float64))


def test_identity_ones_and_transpose():
    rng = np.random.default_rng(2)
    a = rng.standard_normal((9, 9))
    assert np.max(np.abs(G.gemm_nt(a, np.eye(9)) - a)) == 0.0          # A I^T = A (not A^T: catches a swapped operand)
    assert np.all(G.gemm_nt(np.ones((3, 13)), np.ones((4, 13))) == 13.0)
    b = rng.standard_normal((5, 9))
    assert np.max(np.abs(G.gemm_nt(a, b).T - G.gemm_nt(b, a))) < 1e-13
    assert np.max(np.abs(G.gemm_nt_rows(a, b, [2, 7]) - G.gemm_nt(a, b)[[2, 7]])) == 0.0
