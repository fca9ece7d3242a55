"""Separate query / key lengths (sdpa_fwd_varlen_qk, sdpa_bwd_varlen_qk) against the fp64 oracle."""
import numpy as np
import pytest
import torch

import sdpa_testlib as TL
from oracle import varlen_qk as V
from paper_2608_17379_b200 import binding
from paper_2608_17379_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _run(q_lens, k_lens, Hq, Hkv, D, causal, seed):
    cu_q = np.zeros(len(q_lens) + 1, dtype=np.int32); cu_q[1:] = np.cumsum(q_lens)
    cu_k = np.zeros(len(k_lens) + 1, dtype=np.int32); cu_k[1:] = np.cumsum(k_lens)
    Tq, Tk = int(cu_q[-1]), int(cu_k[-1])
    scale = 1.0 / np.sqrt(D)
    qb = W.gen_tensor_bits(seed, W.TENSOR_Q, (Tq, Hq, D))
    kb = W.gen_tensor_bits(seed, W.TENSOR_K, (Tk, Hkv, D))
    vb = W.gen_tensor_bits(seed, W.TENSOR_V, (Tk, Hkv, D))
    dob = W.gen_tensor_bits(seed, W.TENSOR_DO, (Tq, Hq, D))
    q, k, v, do = (TL.to_dev(x) for x in (qb, kb, vb, dob))
    cq, ck = torch.from_numpy(cu_q).cuda(), torch.from_numpy(cu_k).cuda()
    mq, mk = int(max(q_lens)), int(max(k_lens))
    o, lse = binding.sdpa_fwd_varlen_qk(q, k, v, cq, ck, mq, mk, causal, scale)
    dk = torch.full_like(k, 7.0); dv = torch.full_like(v, 7.0)  # every key row must be written
    dq, dk, dv = binding.sdpa_bwd_varlen_qk(q, k, v, o, lse, do, cq, ck, mq, mk, causal, scale, dk=dk, dv=dv)
    torch.cuda.synchronize()
    assert binding.query_status() == (0, 0)
    f = W.bf16_bits_to_f64
    rdq, rdk, rdv, ro, rlse = V.sdpa_bwd_qk(f(qb), f(kb), f(vb), f(dob), cu_q, cu_k, causal, scale)
    assert np.max(np.abs(TL.to_f64(o) - ro)) <= TL.TOL_O
    assert np.max(np.abs(TL.to_f64(lse) - rlse)) <= TL.TOL_LSE
    for got, ref, name in ((dq, rdq, "dq"), (dk, rdk, "dk"), (dv, rdv, "dv")):
        err = np.max(np.abs(TL.to_f64(got) - ref)) / max(np.max(np.abs(ref)), TL.GRAD_FLOOR)
        assert err <= TL.TOL_GRAD, (name, err)


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("q_lens,k_lens,Hq,Hkv,D", [
    ((5,), (9,), 2, 1, 64),
    ((130,), (130,), 2, 2, 128),                    # equal lengths through the new entry points
    ((100, 1, 257), (400, 130, 257), 6, 2, 128),    # more keys than queries
    ((64, 200), (64 + 128, 200 + 300), 4, 2, 128),  # offsets that are and are not multiples of the tile
    ((0, 50, 0), (30, 50, 0), 2, 1, 64),            # keys without queries get zero gradients
    ((300,), (1000,), 4, 1, 96),
])
def test_more_keys_than_queries(q_lens, k_lens, Hq, Hkv, D, causal):
    _run(q_lens, k_lens, Hq, Hkv, D, causal, seed=9500 + len(q_lens) + Hq)


def test_fewer_keys_than_queries_without_mask():
    _run((300, 129), (77, 1), 4, 2, 128, False, seed=9600)


def test_paper_paged_prefill_lengths_packed():
    """The lengths of the paper's paged prefill workload (892 query tokens against longer key histories),
    as packed tensors, with the backward pass."""
    rng = np.random.default_rng(11)
    q_lens = [int(x) for x in rng.multinomial(892, np.ones(7) / 7)]
    k_lens = [ql + int(x) for ql, x in zip(q_lens, rng.integers(0, 900, 7))]
    _run(q_lens, k_lens, 32, 4, 128, True, seed=9700)


def test_causal_with_fewer_keys_than_queries_is_reported():
    q = torch.zeros((10, 2, 64), dtype=torch.bfloat16, device="cuda"); k = torch.zeros((5, 2, 64), dtype=torch.bfloat16, device="cuda")
    cq = torch.tensor([0, 10], dtype=torch.int32, device="cuda"); ck = torch.tensor([0, 5], dtype=torch.int32, device="cuda")
    binding.sdpa_fwd_varlen_qk(q, k, k, cq, ck, 10, 5, True, 0.125)
    torch.cuda.synchronize()
    st, _ = binding.query_status()
    assert st == 2
    assert binding.query_status() == (0, 0)
