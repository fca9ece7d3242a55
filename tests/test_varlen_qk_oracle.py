"""Pins for the oracle with separate query / key lengths (CPU only)."""
import numpy as np

import oracle
from oracle import paged as P
from oracle import varlen_qk as V


def _rand(rng, cu_q, cu_k, Hq, Hkv, D):
    Tq, Tk = int(cu_q[-1]), int(cu_k[-1])
    return (rng.standard_normal((Tq, Hq, D)), rng.standard_normal((Tk, Hkv, D)),
            rng.standard_normal((Tk, Hkv, D)), rng.standard_normal((Tq, Hq, D)))


def test_equal_lengths_reduce_to_the_c_oracle():
    rng = np.random.default_rng(0)
    cu = np.array([0, 7, 7, 19], dtype=np.int32)
    q, k, v, do = _rand(rng, cu, cu, 4, 2, 8)
    for causal in (False, True):
        dq0, dk0, dv0, o0, lse0 = oracle.sdpa_bwd(q, k, v, do, cu, causal, 0.37)
        dq, dk, dv, o, lse = V.sdpa_bwd_qk(q, k, v, do, cu, cu, causal, 0.37)
        for a, b in ((dq, dq0), (dk, dk0), (dv, dv0), (o, o0), (lse, lse0)):
            assert np.max(np.abs(a - b)) < 1e-11


def test_forward_equals_the_paged_oracle_with_an_identity_page_table():
    rng = np.random.default_rng(1)
    cu_q = np.array([0, 3, 8], dtype=np.int32)
    cu_k = np.array([0, 9, 14], dtype=np.int32)
    q, k, v, _ = _rand(rng, cu_q, cu_k, 4, 2, 8)
    for causal in (False, True):
        o0, lse0 = P.sdpa_fwd_paged(q, k, v, cu_q, cu_k, np.arange(14), causal, 0.5)
        o, lse = V.sdpa_fwd_qk(q, k, v, cu_q, cu_k, causal, 0.5)
        assert np.max(np.abs(o - o0)) < 1e-12 and np.max(np.abs(lse - lse0)) < 1e-12


def test_gradients_match_central_finite_differences():
    rng = np.random.default_rng(2)
    cu_q = np.array([0, 2, 5], dtype=np.int32)
    cu_k = np.array([0, 4, 7], dtype=np.int32)   # Lk - Lq = 2 and 0
    q, k, v, do = _rand(rng, cu_q, cu_k, 2, 1, 3)
    eps = 1e-6
    for causal in (False, True):
        dq, dk, dv, _, _ = V.sdpa_bwd_qk(q, k, v, do, cu_q, cu_k, causal, 0.7)
        loss = lambda q_, k_, v_: float(np.sum(do * V.sdpa_fwd_qk(q_, k_, v_, cu_q, cu_k, causal, 0.7)[0]))
        for x, g, which in ((q, dq, 0), (k, dk, 1), (v, dv, 2)):
            it = np.nditer(x, flags=["multi_index"])
            for _ in it:
                idx = it.multi_index
                args_p = [q.copy(), k.copy(), v.copy()]; args_m = [q.copy(), k.copy(), v.copy()]
                args_p[which][idx] += eps; args_m[which][idx] -= eps
                fd = (loss(*args_p) - loss(*args_m)) / (2 * eps)
                assert abs(fd - g[idx]) < 1e-6, (causal, which, idx, fd, g[idx])


def test_causal_alignment_first_and_last_query():
    """With Lq = 2 and Lk = 5 the first query sees keys 0..3 and the last query sees all five."""
    rng = np.random.default_rng(3)
    cu_q = np.array([0, 2], dtype=np.int32); cu_k = np.array([0, 5], dtype=np.int32)
    q, k, v, _ = _rand(rng, cu_q, cu_k, 1, 1, 4)
    o, lse = V.sdpa_fwd_qk(q, k, v, cu_q, cu_k, True, 1.0)
    for i, n in ((0, 4), (1, 5)):
        s = k[:n, 0] @ q[i, 0]
        w = np.exp(s - s.max())
        assert np.max(np.abs(o[i, 0] - (w / w.sum()) @ v[:n, 0])) < 1e-12
        assert abs(lse[0, i] - (s.max() + np.log(w.sum()))) < 1e-12
