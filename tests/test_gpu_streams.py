"""Calls on several streams at once: every call owns its buffers and workspace, so results must equal
the single-stream results bit for bit (forward, dK, dV) or within the dQ tolerance."""
import pytest
import torch

import sdpa_testlib as TL
from paper_2608_17379_b200 import binding
from paper_2608_17379_b200 import workloads as W

pytestmark = pytest.mark.gpu


def test_concurrent_streams_match_serial_results():
    ws = [TL.random_workload((400 + 50 * i, 129), 4, 2, 128, bool(i & 1), seed=900 + i) for i in range(4)]
    data = []
    for w in ws:
        qb, kb, vb, dob = W.make_inputs(w)
        data.append([TL.to_dev(x) for x in (qb, kb, vb, dob)] + [torch.from_numpy(w.cu_seqlens).cuda()])
    ref = []
    for w, (q, k, v, do, cu) in zip(ws, data):
        o, lse = binding.sdpa_fwd(q, k, v, cu, w.max_seqlen, w.causal, w.scale)
        ref.append((o, lse) + binding.sdpa_bwd(q, k, v, o, lse, do, cu, w.max_seqlen, w.causal, w.scale))
    torch.cuda.synchronize()
    streams = [torch.cuda.Stream() for _ in ws]
    got = []
    for _ in range(3):  # a few rounds so that launches really overlap
        got = []
        for w, (q, k, v, do, cu), st in zip(ws, data, streams):
            with torch.cuda.stream(st):
                o, lse = binding.sdpa_fwd(q, k, v, cu, w.max_seqlen, w.causal, w.scale, stream=st)
                got.append((o, lse) + binding.sdpa_bwd(q, k, v, o, lse, do, cu, w.max_seqlen, w.causal, w.scale, stream=st))
    torch.cuda.synchronize()
    assert binding.query_status() == (0, 0)
    for a, b in zip(ref, got):
        assert torch.equal(a[0].view(torch.int16), b[0].view(torch.int16))
        assert torch.equal(a[1], b[1])
        assert torch.equal(a[3].view(torch.int16), b[3].view(torch.int16))
        assert torch.equal(a[4].view(torch.int16), b[4].view(torch.int16))
        assert (a[2].float() - b[2].float()).abs().max().item() <= 2e-2 * a[2].float().abs().max().item()
