"""fp64 CPU oracle for the bf16 GEMM C = A B^T.

TEST INFRASTRUCTURE ONLY (tests, smoke check, bench's CPU legs); never imported by the product path.
The operation (paper, appendix "Workloads": C = A B^T with A [M,K], B [N,K], C [M,N]) has a plain
definition, c_ij = sum_k a_ik b_jk, so the oracle is that definition evaluated in float64 with
numpy's matmul as the library step.  Pins (tests/test_gemm_oracle.py): a pure-Python triple loop on
tiny inputs, exact integer arithmetic, identity and all-ones closed forms, and (A B^T)^T = B A^T.
"""
from __future__ import annotations

import numpy as np


def gemm_nt(a: np.ndarray, b: np.ndarray) -> np.ndarray:
    """a [M,K], b [N,K] -> float64 [M,N] with c[i,j] = sum_k a[i,k] * b[j,k]."""
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    assert a.ndim == 2 and b.ndim == 2 and a.shape[1] == b.shape[1]
    return a @ b.T


def gemm_nt_rows(a: np.ndarray, b: np.ndarray, rows) -> np.ndarray:
    """Only the listed output rows (for sampled checks of large products)."""
    return gemm_nt(np.asarray(a, dtype=np.float64)[list(rows)], b)
