"""sdpa_decode_paged (one query token per sequence, split keys, GQA rows packed into the tile) against the
fp64 paged oracle, and against sdpa_fwd_paged on the same inputs."""
import numpy as np
import pytest
import torch

import sdpa_testlib as TL
from oracle import paged as P
from paper_2608_17379_b200 import binding
from paper_2608_17379_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _run(k_lens, Hq, Hkv, D, num_pages, seed):
    rng = np.random.default_rng(seed)
    B = len(k_lens)
    cu = np.arange(B + 1, dtype=np.int32)
    indptr = np.concatenate([[0], np.cumsum(k_lens)]).astype(np.int32)
    idx = rng.choice(num_pages, int(sum(k_lens)), replace=False).astype(np.int32)
    qb = W.gen_tensor_bits(seed, W.TENSOR_Q, (B, Hq, D))
    kb = W.gen_tensor_bits(seed, W.TENSOR_K, (num_pages, Hkv, D))
    vb = W.gen_tensor_bits(seed, W.TENSOR_V, (num_pages, Hkv, D))
    scale = 1.0 / np.sqrt(D)
    q, kc, vc = TL.to_dev(qb), TL.to_dev(kb), TL.to_dev(vb)
    ip, ix = torch.from_numpy(indptr).cuda(), torch.from_numpy(idx).cuda()
    o, lse = binding.sdpa_decode_paged(q, kc, vc, ip, ix, int(max(k_lens)), scale)
    torch.cuda.synchronize()
    assert binding.query_status() == (0, 0)
    o_ref, lse_ref = P.sdpa_fwd_paged(W.bf16_bits_to_f64(qb), W.bf16_bits_to_f64(kb), W.bf16_bits_to_f64(vb), cu, indptr,
                                      idx, True, scale)
    assert np.max(np.abs(TL.to_f64(o) - o_ref)) <= TL.TOL_O
    assert np.max(np.abs(TL.to_f64(lse) - lse_ref)) <= TL.TOL_LSE
    # the general paged kernel on the same problem (different tiling and split: equal up to rounding)
    o2, lse2 = binding.sdpa_fwd_paged(q, kc, vc, torch.from_numpy(cu).cuda(), ip, ix, 1, True, scale)
    assert (o.float() - o2.float()).abs().max().item() <= 2e-2
    assert (lse - lse2).abs().max().item() <= 1e-3


@pytest.mark.parametrize("k_lens,Hq,Hkv,D", [
    ((5,), 2, 1, 64),
    ((1, 128, 129), 4, 4, 128),          # G = 1
    ((300, 77, 1000), 8, 2, 128),        # G = 4, ragged splits
    ((2000, 3, 700, 129), 32, 4, 128),   # G = 8
    ((640,) * 6, 24, 8, 96),             # G = 3, padded head dimension
    ((50,) * 40, 64, 1, 64),             # G = 64: two warps of the tile hold heads
])
def test_decode_shapes(k_lens, Hq, Hkv, D):
    _run(k_lens, Hq, Hkv, D, num_pages=int(sum(k_lens)) + 101, seed=9800 + Hq)


def test_paper_decode_shape():
    """Batch 15, one query token each, 9,625 KV-page indices in total, 42,784-page cache, 24 / 8 heads."""
    rng = np.random.default_rng(5)
    cuts = np.sort(rng.choice(np.arange(1, 9625), 14, replace=False))
    k_lens = [int(x) for x in np.diff(np.concatenate([[0], cuts, [9625]]))]
    _run(k_lens, 24, 8, 128, num_pages=42784, seed=9900)


def test_bad_page_index_is_reported():
    qb = W.gen_tensor_bits(1, W.TENSOR_Q, (1, 2, 64)); kb = W.gen_tensor_bits(1, W.TENSOR_K, (16, 2, 64))
    ip = torch.tensor([0, 8], dtype=torch.int32, device="cuda")
    idx = torch.tensor([0, 1, 2, 3, 99, 5, 6, 7], dtype=torch.int32, device="cuda")
    binding.sdpa_decode_paged(TL.to_dev(qb), TL.to_dev(kb), TL.to_dev(kb), ip, idx, 8, 0.1)
    torch.cuda.synchronize()
    assert binding.query_status()[0] == 2
