"""sdpa_bwd_deterministic: bit-identical gradients from run to run, and the same values as sdpa_bwd up to
the order of the fp32 additions of dq."""
import numpy as np
import pytest
import torch

import sdpa_testlib as TL
from paper_2608_17379_b200 import binding
from paper_2608_17379_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _grads(w, deterministic, repeats):
    inputs = W.make_inputs(w)
    q, k, v, do = (TL.to_dev(x) for x in inputs)
    cu = torch.from_numpy(w.cu_seqlens).cuda()
    o, lse = binding.sdpa_fwd(q, k, v, cu, w.max_seqlen, w.causal, w.scale)
    outs = []
    for _ in range(repeats):
        outs.append(binding.sdpa_bwd(q, k, v, o, lse, do, cu, w.max_seqlen, w.causal, w.scale,
                                     deterministic=deterministic))
    torch.cuda.synchronize()
    assert binding.query_status() == (0, 0)
    return inputs, dict(o=o, lse=lse), outs


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("lengths,Hq,Hkv,D", [
    ((700,), 2, 1, 128),
    ((300, 77, 0, 513), 4, 2, 128),
    ((1000, 130), 8, 1, 64),
    ((2048,) * 2, 8, 2, 128),      # 16 key tiles taking turns
])
def test_three_runs_are_bit_identical_and_correct(lengths, Hq, Hkv, D, causal):
    w = TL.random_workload(lengths, Hq, Hkv, D, causal, seed=9100 + Hq + D)
    inputs, fwd, outs = _grads(w, True, 3)
    for other in outs[1:]:
        for a, b in zip(outs[0], other):
            assert torch.equal(a.view(torch.int16), b.view(torch.int16))
    dq, dk, dv = outs[0]
    worst = TL.compare_slices(w, inputs, dict(fwd, dq=dq, dk=dk, dv=dv), TL.all_slices(w))
    TL.assert_within(worst)
    # against the default mode: dk and dv are accumulated inside one CTA in the same order in both modes
    # (bit-identical); dq is the same sum in another order
    _, _, plain = _grads(w, False, 1)
    assert torch.equal(plain[0][1].view(torch.int16), dk.view(torch.int16))
    assert torch.equal(plain[0][2].view(torch.int16), dv.view(torch.int16))
    a, b = plain[0][0].float(), dq.float()
    assert (a - b).abs().max().item() <= 2e-2 * max(a.abs().max().item(), 1e-2)


def test_bench_workload_twice():
    w = W.config("c3")
    _, _, outs = _grads(w, True, 2)
    for a, b in zip(outs[0], outs[1]):
        assert torch.equal(a.view(torch.int16), b.view(torch.int16))
