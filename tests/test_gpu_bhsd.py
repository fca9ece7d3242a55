"""Dense [B, H, S, D] entry points: they must compute what the packed entry points compute, on the same
values laid out the other way round, and leave the rows past a sequence's length alone."""
import numpy as np
import pytest
import torch

import sdpa_testlib as TL
from paper_2608_17379_b200 import binding
from paper_2608_17379_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _to_dense(packed, w, S, fill):
    """[T, H, D] packed rows -> [B, H, S, D]; rows past a sequence's length hold `fill`."""
    T, H, D = packed.shape
    out = torch.full((w.B, H, S, D), fill, dtype=packed.dtype, device=packed.device)
    cu = w.cu_seqlens
    for b in range(w.B):
        L = int(cu[b + 1] - cu[b])
        out[b, :, :L] = packed[cu[b]:cu[b + 1]].permute(1, 0, 2)
    return out.contiguous()


def _from_dense(dense, w):
    cu = w.cu_seqlens
    parts = [dense[b, :, :int(cu[b + 1] - cu[b])].permute(1, 0, 2) for b in range(w.B)]
    return torch.cat(parts, dim=0).contiguous()


def _run_both(w, S, with_lengths):
    inputs = W.make_inputs(w)
    q, k, v, do = (TL.to_dev(x) for x in inputs)
    cu = torch.from_numpy(w.cu_seqlens).cuda()
    o, lse = binding.sdpa_fwd(q, k, v, cu, w.max_seqlen, w.causal, w.scale)
    dq, dk, dv = binding.sdpa_bwd(q, k, v, o, lse, do, cu, w.max_seqlen, w.causal, w.scale)
    # padding rows: finite values that would be visible in the results if they were used
    qd, kd, vd, dod = (_to_dense(x, w, S, 3.0) for x in (q, k, v, do))
    canary = 1024.0  # exactly representable in bf16
    od = torch.full_like(qd, canary)
    lsed = torch.full((w.B, w.Hq, S), canary, dtype=torch.float32, device="cuda")
    dqd, dkd, dvd = torch.full_like(qd, canary), torch.full_like(kd, canary), torch.full_like(vd, canary)
    cu_arg = cu if with_lengths else None
    binding.sdpa_fwd_bhsd(qd, kd, vd, w.causal, w.scale, cu_seqlens=cu_arg, o=od, lse=lsed)
    binding.sdpa_bwd_bhsd(qd, kd, vd, od, lsed, dod, w.causal, w.scale, cu_seqlens=cu_arg, dq=dqd, dk=dkd, dv=dvd)
    assert binding.query_status() == (0, 0)
    packed = dict(o=o, lse=lse, dq=dq, dk=dk, dv=dv)
    dense = dict(o=od, lse=lsed, dq=dqd, dk=dkd, dv=dvd)
    return inputs, packed, dense, canary


def _check_same(w, packed, dense):
    # same tiles, same order of operations: everything but the atomically accumulated dq is bit-identical
    for name in ("o", "dk", "dv"):
        got = _from_dense(dense[name], w)
        assert torch.equal(got.view(torch.int16), packed[name].view(torch.int16)), name
    cu = w.cu_seqlens
    for b in range(w.B):
        L = int(cu[b + 1] - cu[b])
        assert torch.equal(dense["lse"][b, :, :L], packed["lse"][:, cu[b]:cu[b + 1]])
    dq = _from_dense(dense["dq"], w).float()
    ref = packed["dq"].float()
    assert (dq - ref).abs().max().item() <= 2e-2 * max(ref.abs().max().item(), 1e-2)


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("Hq,Hkv,D", [(4, 2, 128), (2, 2, 64), (3, 1, 96)])
def test_full_length_dense_equals_packed(Hq, Hkv, D, causal):
    w = TL.random_workload((300, 300), Hq, Hkv, D, causal, seed=8100 + D + Hq)
    inputs, packed, dense, _ = _run_both(w, 300, with_lengths=False)
    _check_same(w, packed, dense)
    worst = TL.compare_slices(w, inputs, packed, TL.all_slices(w))
    TL.assert_within(worst)


@pytest.mark.parametrize("causal", [False, True])
def test_dense_with_lengths_leaves_padding_rows_alone(causal):
    w = TL.random_workload((300, 77, 0, 513), 4, 2, 128, causal, seed=8200)
    S = 520
    _, packed, dense, canary = _run_both(w, S, with_lengths=True)
    _check_same(w, packed, dense)
    cu = w.cu_seqlens
    for b in range(w.B):
        L = int(cu[b + 1] - cu[b])
        for name in ("o", "dk", "dv"):
            assert bool((dense[name][b, :, L:].float() == canary).all()), (name, b)
        assert bool((dense["lse"][b, :, L:] == canary).all())
        assert bool((dense["dq"][b, :, L:].float() == 0).all())


def test_paper_shape_dense_sampled():
    """[4, 48, 4096, 128]-shaped call at a quarter of the heads (appendix "Workloads"): sampled slices
    against the oracle."""
    w = TL.random_workload((4096,) * 4, 12, 12, 128, True, seed=8300)
    inputs, packed, dense, _ = _run_both(w, 4096, with_lengths=False)
    _check_same(w, packed, dense)
    worst = TL.compare_slices(w, inputs, packed, [(0, 0), (3, 11)])
    TL.assert_within(worst)
