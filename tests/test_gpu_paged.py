"""Parity of sdpa_fwd_paged (through the C ABI) against the fp64 paged oracle; tolerances as for sdpa_fwd."""
import numpy as np
import pytest
import torch

import sdpa_testlib as TL
from oracle import paged as P
from paper_2608_17379_b200 import binding
from paper_2608_17379_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _run(q_lens, k_lens, Hq, Hkv, D, num_pages, causal, seed):
    rng = np.random.default_rng(seed)
    Tq = int(sum(q_lens))
    cu = np.concatenate([[0], np.cumsum(q_lens)]).astype(np.int32)
    indptr = np.concatenate([[0], np.cumsum(k_lens)]).astype(np.int32)
    idx = rng.choice(num_pages, int(sum(k_lens)), replace=False).astype(np.int32)
    qb = W.gen_tensor_bits(seed, W.TENSOR_Q, (Tq, Hq, D))
    kb = W.gen_tensor_bits(seed, W.TENSOR_K, (num_pages, Hkv, D))
    vb = W.gen_tensor_bits(seed, W.TENSOR_V, (num_pages, Hkv, D))
    scale = 1.0 / np.sqrt(D)
    o, lse = binding.sdpa_fwd_paged(TL.to_dev(qb), TL.to_dev(kb), TL.to_dev(vb), torch.from_numpy(cu).cuda(),
                                    torch.from_numpy(indptr).cuda(), torch.from_numpy(idx).cuda(), int(max(q_lens)),
                                    causal, scale)
    assert binding.query_status() == (0, 0)
    o_ref, lse_ref = P.sdpa_fwd_paged(W.bf16_bits_to_f64(qb), W.bf16_bits_to_f64(kb), W.bf16_bits_to_f64(vb), cu, indptr,
                                      idx, causal, scale)
    assert np.max(np.abs(TL.to_f64(o) - o_ref)) <= TL.TOL_O
    assert np.max(np.abs(TL.to_f64(lse) - lse_ref)) <= TL.TOL_LSE


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("q_lens,k_lens,Hq,Hkv,D", [
    ((5,), (5,), 2, 1, 64),
    ((130,), (130,), 2, 2, 128),
    ((300, 77), (300, 77), 4, 2, 128),
    ((100, 1, 257), (400, 130, 257), 6, 2, 128),   # more keys than queries: end-aligned causal mask
    ((90, 200), (300, 200), 4, 2, 96),             # head dimension between the kernels: zero-padded columns
    ((33,), (140,), 2, 1, 40),
])
def test_small_paged_shapes(q_lens, k_lens, Hq, Hkv, D, causal):
    _run(q_lens, k_lens, Hq, Hkv, D, num_pages=int(sum(k_lens)) + 37, causal=causal, seed=300 + len(q_lens) + Hq)


def test_paper_paged_prefill_shape():
    """24 query / 8 KV heads, D=128, page size 1, one sequence of 892 query tokens and 892 KV pages in a
    43,676-page cache (page numbers synthetic)."""
    _run((892,), (892,), 24, 8, 128, num_pages=43676, causal=True, seed=401)


def test_paper_paged_decode_shape():
    """Batch 15, one query token each, 9,625 KV-page indices in total, 42,784-page cache."""
    rng = np.random.default_rng(5)
    cuts = np.sort(rng.choice(np.arange(1, 9625), 14, replace=False))
    k_lens = np.diff(np.concatenate([[0], cuts, [9625]]))
    _run((1,) * 15, tuple(int(x) for x in k_lens), 24, 8, 128, num_pages=42784, causal=True, seed=402)


def test_bad_page_index_is_reported():
    qb = W.gen_tensor_bits(1, W.TENSOR_Q, (8, 2, 64)); kb = W.gen_tensor_bits(1, W.TENSOR_K, (16, 2, 64))
    cu = torch.tensor([0, 8], dtype=torch.int32, device="cuda")
    idx = torch.tensor([0, 1, 2, 3, 99, 5, 6, 7], dtype=torch.int32, device="cuda")
    binding.sdpa_fwd_paged(TL.to_dev(qb), TL.to_dev(kb), TL.to_dev(kb), cu, cu, idx, 8, True, 0.1)
    assert binding.query_status()[0] == 2
