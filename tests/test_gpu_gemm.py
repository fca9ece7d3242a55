"""Parity of the bf16 GEMM kernel (through the C ABI) against the fp64 oracle.

Tolerance: |c - c*| <= 1e-2 * (1 + |c*|) element-wise (the benchmark's allclose(atol=rtol=1e-2)):
the output is rounded once to bf16 (2^-9 relative) after an fp32 accumulation over K."""
import numpy as np
import pytest
import torch

import sdpa_testlib as TL
from oracle import gemm as G
from paper_2608_17379_b200 import binding
from paper_2608_17379_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _inputs(M, N, K, seed):
    a = W.gen_tensor_bits(seed, W.TENSOR_Q, (M, K))
    b = W.gen_tensor_bits(seed, W.TENSOR_K, (N, K))
    return a, b


def _close(got, ref):
    return np.all(np.abs(got - ref) <= 1e-2 * (1.0 + np.abs(ref)))


@pytest.mark.parametrize("M,N,K", [(128, 224, 64), (1, 8, 8), (130, 232, 72), (257, 456, 200), (512, 1000, 1024),
                                   (1000, 64, 4096), (128 * 3 + 5, 224 * 2 + 16, 64 * 7 + 8)])
def test_small_and_ragged_shapes(M, N, K):
    a, b = _inputs(M, N, K, 200 + M)
    c = binding.gemm_bf16_nt(TL.to_dev(a), TL.to_dev(b))
    assert binding.query_status() == (0, 0)
    ref = G.gemm_nt(W.bf16_bits_to_f64(a), W.bf16_bits_to_f64(b))
    assert _close(TL.to_f64(c), ref)


def test_paper_shape_sampled_rows_and_bit_reproducibility():
    """8192 x 7168 x 5120: 48 sampled rows of C against the oracle; two runs are bit-identical."""
    M, N, K = 8192, 7168, 5120
    a, b = _inputs(M, N, K, 7)
    ad, bd = TL.to_dev(a), TL.to_dev(b)
    c1 = binding.gemm_bf16_nt(ad, bd)
    c2 = binding.gemm_bf16_nt(ad, bd)
    assert binding.query_status() == (0, 0)
    assert torch.equal(c1.view(torch.int16), c2.view(torch.int16))
    rows = sorted(set(np.random.default_rng(3).integers(0, M, 44).tolist() + [0, 127, 128, M - 1]))
    ref = G.gemm_nt_rows(W.bf16_bits_to_f64(a), W.bf16_bits_to_f64(b), rows)
    assert _close(TL.to_f64(c1[rows]), ref)


def test_output_canaries_and_argument_checks():
    M, N, K = 200, 240, 136
    a, b = _inputs(M, N, K, 9)
    buf = torch.full((M * N + 2048,), -7.0, dtype=torch.bfloat16, device="cuda")
    c = buf[1024:1024 + M * N].view(M, N)
    binding.gemm_bf16_nt(TL.to_dev(a), TL.to_dev(b), c=c)
    assert binding.query_status() == (0, 0)
    assert bool((buf[:1024] == -7.0).all()) and bool((buf[-1024:] == -7.0).all())
    lib = binding.load()
    p = c.data_ptr()
    assert lib.gemm_bf16_nt(p, p, p, 8, 12, 8, None) == -3     # N not a multiple of 8
    assert lib.gemm_bf16_nt(p, p, p, 8, 8, 4, None) == -3      # K not a multiple of 8
    assert lib.gemm_bf16_nt(0, p, p, 8, 8, 8, None) == -1
    assert lib.gemm_bf16_nt(p, p, p, 0, 8, 8, None) == 0       # empty output: no-op
