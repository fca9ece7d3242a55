"""Pins for the paged-attention oracle (CPU only)."""
import math

import numpy as np

import oracle
from oracle import paged as P


def test_identity_page_table_equals_dense_oracle():
    rng = np.random.default_rng(0)
    lengths = [7, 12]
    cu = np.array([0, 7, 19], dtype=np.int32)
    q = rng.standard_normal((19, 4, 8)); k = rng.standard_normal((19, 2, 8)); v = rng.standard_normal((19, 2, 8))
    for causal in (False, True):
        o_ref, lse_ref = oracle.sdpa_fwd(q, k, v, cu, causal, 0.4)
        o, lse = P.sdpa_fwd_paged(q, k, v, cu, cu, np.arange(19), causal, 0.4)
        assert np.max(np.abs(o - o_ref)) < 1e-12 and np.max(np.abs(lse - lse_ref)) < 1e-12


def test_scattered_pages_and_python_loop():
    rng = np.random.default_rng(1)
    Pn, Hq, Hkv, D = 23, 2, 1, 4
    kc = rng.standard_normal((Pn, Hkv, D)); vc = rng.standard_normal((Pn, Hkv, D))
    q = rng.standard_normal((3, Hq, D))
    cu = np.array([0, 3]); indptr = np.array([0, 5]); idx = np.array([17, 2, 9, 22, 4])
    o, lse = P.sdpa_fwd_paged(q, kc, vc, cu, indptr, idx, True, 0.5)
    for i in range(3):
        for h in range(Hq):
            keys = idx[: i + 3]  # end-aligned: query i of 3 sees keys 0 .. i + 2
            s = [0.5 * sum(q[i, h, d] * kc[p, 0, d] for d in range(D)) for p in keys]
            w = [math.exp(x) for x in s]
            ref = [sum(wj * vc[p, 0, d] for wj, p in zip(w, keys)) / sum(w) for d in range(D)]
            assert np.max(np.abs(o[i, h] - np.array(ref))) < 1e-12
            assert abs(lse[h, i] - math.log(sum(w))) < 1e-12


def test_decode_row_sees_every_key():
    rng = np.random.default_rng(2)
    kc = rng.standard_normal((40, 2, 8)); vc = np.ones((40, 2, 8)) * np.arange(8)
    q = np.zeros((2, 4, 8))  # two sequences, one query each, q = 0 -> uniform average, lse = ln Lk
    cu = np.array([0, 1, 2]); indptr = np.array([0, 10, 35]); idx = rng.permutation(40)[:35]
    o, lse = P.sdpa_fwd_paged(q, kc, vc, cu, indptr, idx, True, 1.0)
    assert np.max(np.abs(o - np.arange(8))) < 1e-12
    assert np.max(np.abs(lse[:, 0] - math.log(10))) < 1e-12 and np.max(np.abs(lse[:, 1] - math.log(25))) < 1e-12
