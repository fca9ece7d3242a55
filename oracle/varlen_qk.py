"""fp64 CPU oracle for attention with separate query and key lengths per sequence (forward and backward).

TEST INFRASTRUCTURE ONLY.  Plain definition: sequence b has Lq_b query rows (cu_q) and Lk_b key/value rows
(cu_k) in packed tensors; query i attends to keys 0 .. i + (Lk - Lq) when causal (the last query sees the
last key: the alignment the paper's paged prefill workload uses, appendix "Generalization attention
workloads"), to all Lk keys otherwise.  Forward: O = softmax(scale q k^T) v, LSE = log sum exp of the
scaled, masked scores.  Backward, for the loss sum(dO * O): P = softmax, dV = P^T dO, dP = dO V^T,
D_i = rowsum(dO * O), dS = P * (dP - D), dQ = scale dS K, dK = scale dS^T Q, summed over the query heads of
a kv head.  Written with numpy in float64, one (sequence, head) at a time, materialised scores, no tiling.
Pins (tests/test_varlen_qk_oracle.py): equality with the C oracle when the lengths are equal, central
finite differences of the forward pass, the forward pass against the paged oracle with an identity page
table, and the mask's first and last rows.
"""
from __future__ import annotations

import numpy as np


def _allowed(Lq: int, Lk: int, causal: bool) -> np.ndarray:
    if not causal:
        return np.ones((Lq, Lk), dtype=bool)
    return np.arange(Lk)[None, :] <= (np.arange(Lq)[:, None] + (Lk - Lq))


def sdpa_fwd_qk(q, k, v, cu_q, cu_k, causal: bool, scale: float):
    """q [Tq,Hq,D], k,v [Tk,Hkv,D] -> (o [Tq,Hq,D], lse [Hq,Tq]) in float64."""
    o, lse, _ = _forward(q, k, v, cu_q, cu_k, causal, scale)
    return o, lse


def _forward(q, k, v, cu_q, cu_k, causal, scale):
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    Tq, Hq, D = q.shape
    G = Hq // k.shape[1]
    o = np.zeros_like(q)
    lse = np.zeros((Hq, Tq))
    probs = {}
    for b in range(len(cu_q) - 1):
        r0, r1 = int(cu_q[b]), int(cu_q[b + 1])
        c0, c1 = int(cu_k[b]), int(cu_k[b + 1])
        if r1 == r0:
            continue
        allowed = _allowed(r1 - r0, c1 - c0, causal)
        assert allowed.any(axis=1).all(), "a query row without a visible key"
        for h in range(Hq):
            s = scale * (q[r0:r1, h] @ k[c0:c1, h // G].T)
            s = np.where(allowed, s, -np.inf)
            m = s.max(axis=1, keepdims=True)
            e = np.exp(s - m)
            l = e.sum(axis=1, keepdims=True)
            p = e / l
            probs[(b, h)] = p
            o[r0:r1, h] = p @ v[c0:c1, h // G]
            lse[h, r0:r1] = (m + np.log(l))[:, 0]
    return o, lse, probs


def sdpa_bwd_qk(q, k, v, dout, cu_q, cu_k, causal: bool, scale: float):
    """Returns (dq, dk, dv, o, lse) in float64 for the loss sum(dout * o)."""
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    dout = np.asarray(dout, dtype=np.float64)
    o, lse, probs = _forward(q, k, v, cu_q, cu_k, causal, scale)
    Hq = q.shape[1]
    G = Hq // k.shape[1]
    dq = np.zeros_like(q)
    dk = np.zeros_like(k)
    dv = np.zeros_like(v)
    for (b, h), p in probs.items():
        r0, r1 = int(cu_q[b]), int(cu_q[b + 1])
        c0, c1 = int(cu_k[b]), int(cu_k[b + 1])
        g = h // G
        do = dout[r0:r1, h]
        dv[c0:c1, g] += p.T @ do
        dp = do @ v[c0:c1, g].T
        delta = np.sum(do * o[r0:r1, h], axis=1, keepdims=True)
        ds = p * (dp - delta)
        dq[r0:r1, h] = scale * (ds @ k[c0:c1, g])
        dk[c0:c1, g] += scale * (ds.T @ q[r0:r1, h])
    return dq, dk, dv, o, lse
