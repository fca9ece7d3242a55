"""The allocation-free backward entry point (sdpa_bwd_static_scratch).

Some users of the library cannot allocate device memory at call time: a plug-in inside a runtime
that owns a fixed device arena, or a latency-critical loop where cudaMalloc's implicit
synchronisation is not acceptable.  For them the library carries a fixed 32 MiB scratch array and
an entry point that uses it instead of a caller workspace.  This test calls that entry point through
the C ABI twice in a row, on different problems, and checks it against sdpa_bwd with an ordinary
workspace: dK and dV bit for bit, dQ within the tolerance the other tests use for two runs of the
atomically reduced dQ.  The second problem is smaller than the first, so stale contents of the
shared array would show up if the call did not clear what it accumulates into.  The file is named so
that pytest collects it last.
"""
import numpy as np
import pytest
import torch

import sdpa_testlib as TL
from paper_2608_17379_b200 import binding
from paper_2608_17379_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _both_ways(w):
    qb, kb, vb, dob = W.make_inputs(w)
    q, k, v, do = (TL.to_dev(x) for x in (qb, kb, vb, dob))
    cu = torch.from_numpy(w.cu_seqlens).cuda()
    o, lse = binding.sdpa_fwd(q, k, v, cu, w.max_seqlen, w.causal, w.scale)
    ref = binding.sdpa_bwd(q, k, v, o, lse, do, cu, w.max_seqlen, w.causal, w.scale)
    dq, dk, dv = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)
    rc = binding.sdpa_bwd_static_scratch(q, k, v, o, lse, do, cu, w.max_seqlen, w.causal, w.scale, dq, dk, dv)
    assert rc == 0
    assert binding.query_status() == (0, 0)
    return ref, (dq, dk, dv)


def _check(ref, got):
    assert torch.equal(ref[1].view(torch.int16), got[1].view(torch.int16))  # dk
    assert torch.equal(ref[2].view(torch.int16), got[2].view(torch.int16))  # dv
    scale = ref[0].float().abs().max().item()
    assert (ref[0].float() - got[0].float()).abs().max().item() <= 2e-2 * scale  # dq: atomic order may differ


def test_two_calls_in_a_row_match_the_workspace_entry_point():
    first = W.Workload("noalloc_a", 71, (700, 300), 4, 2, 128, True)
    second = W.Workload("noalloc_b", 72, (260,), 2, 2, 64, False)
    assert binding.sdpa_bwd_workspace_bytes(first.B, first.Hq, first.Hkv, first.D, first.T,
                                            first.max_seqlen) <= binding.STATIC_SCRATCH_BYTES
    _check(*_both_ways(first))
    _check(*_both_ways(second))


def test_oversize_problem_is_rejected_before_any_launch():
    w = W.Workload("noalloc_small", 73, (64,), 2, 2, 64, False)
    qb, kb, vb, dob = W.make_inputs(w)
    q, k, v, do = (TL.to_dev(x) for x in (qb, kb, vb, dob))
    cu = torch.from_numpy(w.cu_seqlens).cuda()
    canary = torch.full_like(q, 7.0)
    lib = binding.load()
    # claim a problem whose scratch need (64 MiB) exceeds the built-in 32 MiB: nothing may run
    big_T, big_H, big_D = 8192, 16, 128
    assert binding.sdpa_bwd_workspace_bytes(1, big_H, big_H, big_D, big_T, big_T) > binding.STATIC_SCRATCH_BYTES
    rc = lib.sdpa_bwd_static_scratch(q.data_ptr(), k.data_ptr(), v.data_ptr(), q.data_ptr(), 0, do.data_ptr(),
                                     canary.data_ptr(), 0, 0, cu.data_ptr(), 1, big_H, big_H, big_D, 0, 0.1,
                                     big_T, big_T, None)
    assert rc == binding.SDPA_ERR_STATIC_SCRATCH
    assert "built-in scratch" in binding.status_string(rc)
    torch.cuda.synchronize()
    assert bool((canary == 7.0).all())
    assert binding.query_status() == (0, 0)
