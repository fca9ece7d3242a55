"""fp64 CPU oracle for attention over a paged KV cache with end-aligned causal masking.

TEST INFRASTRUCTURE ONLY.  Plain definition (paper, appendix "Generalization attention workloads":
paged causal prefill / paged decode, page size 1): the keys and values of sequence b are the cache
rows listed in its page table; query i of Lq attends to keys 0 .. i + (Lk - Lq) when causal, to all Lk
keys otherwise; O = softmax(scale q k^T) v, LSE = log sum exp of the scaled, masked scores.  Written
with numpy in float64, one (sequence, head) at a time, no tiling.  Pins (tests/test_paged_oracle.py):
equality with the C oracle when Lk = Lq and the page table is the identity, a pure-Python loop on tiny
inputs, decode rows as plain softmax averages.
"""
from __future__ import annotations

import numpy as np


def sdpa_fwd_paged(q, k_cache, v_cache, cu_q, kv_indptr, kv_indices, causal: bool, scale: float):
    """q [Tq,Hq,D], caches [P,Hkv,D] -> (o [Tq,Hq,D], lse [Hq,Tq]) in float64."""
    q = np.asarray(q, dtype=np.float64)
    k_cache = np.asarray(k_cache, dtype=np.float64)
    v_cache = np.asarray(v_cache, dtype=np.float64)
    Tq, Hq, D = q.shape
    Hkv = k_cache.shape[1]
    G = Hq // Hkv
    o = np.zeros_like(q)
    lse = np.zeros((Hq, Tq))
    for b in range(len(cu_q) - 1):
        r0, r1 = int(cu_q[b]), int(cu_q[b + 1])
        pages = np.asarray(kv_indices[int(kv_indptr[b]):int(kv_indptr[b + 1])], dtype=np.int64)
        Lq, Lk = r1 - r0, len(pages)
        if Lq == 0:
            continue
        assert Lk >= Lq
        if causal:
            allowed = np.arange(Lk)[None, :] <= (np.arange(Lq)[:, None] + (Lk - Lq))
        else:
            allowed = np.ones((Lq, Lk), dtype=bool)
        for h in range(Hq):
            k = k_cache[pages, h // G]
            v = v_cache[pages, h // G]
            s = scale * (q[r0:r1, h] @ k.T)
            s = np.where(allowed, s, -np.inf)
            m = s.max(axis=1, keepdims=True)
            e = np.exp(s - m)
            l = e.sum(axis=1, keepdims=True)
            o[r0:r1, h] = (e / l) @ v
            lse[h, r0:r1] = (m + np.log(l))[:, 0]
    return o, lse
