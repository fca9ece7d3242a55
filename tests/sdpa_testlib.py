"""Shared helpers of the GPU parity tests: run the CUDA path through the C-ABI binding, run the
fp64 oracle on whole tensors or on independent (sequence, kv-head) slices, and compare."""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2608_17379_b200 import binding
from paper_2608_17379_b200 import workloads as W

# Tolerances of the benchmark definition (bf16 path against the unrounded fp64 oracle).
TOL_O = 2e-2      # max |O - O*|
TOL_LSE = 1e-3    # max |LSE - LSE*|
TOL_GRAD = 5e-2   # max |dX - dX*| / max |dX*|
GRAD_FLOOR = 1e-2  # denominator floor for gradients that are exactly zero


def to_dev(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def to_f64(t: torch.Tensor) -> np.ndarray:
    if t.dtype == torch.bfloat16:
        return t.float().cpu().numpy().astype(np.float64)
    return t.cpu().numpy().astype(np.float64)


def run_gpu(qb, kb, vb, dob, cu, max_seqlen, causal, scale, bwd=True):
    """bf16 bit-pattern arrays -> dict of device outputs (torch tensors)."""
    q, k, v, do = (to_dev(x) for x in (qb, kb, vb, dob))
    cu_d = torch.from_numpy(np.ascontiguousarray(cu, dtype=np.int32)).cuda()
    o, lse = binding.sdpa_fwd(q, k, v, cu_d, max_seqlen, causal, scale)
    out = {"o": o, "lse": lse}
    if bwd:
        dq, dk, dv = binding.sdpa_bwd(q, k, v, o, lse, do, cu_d, max_seqlen, causal, scale)
        out.update(dq=dq, dk=dk, dv=dv)
    st, site = binding.query_status()
    assert st == 0, f"device status {st} ({binding.status_string(st)}) at site {site}"
    return out


def compare_slices(w: W.Workload, inputs, gpu_out, slices):
    """Oracle on each (b, g) slice; returns dict name -> worst error over the slices."""
    qb, kb, vb, dob = inputs
    G = w.Hq // w.Hkv
    worst = {"o": 0.0, "lse": 0.0, "dq": 0.0, "dk": 0.0, "dv": 0.0}
    for (b, g) in slices:
        r0, r1, h0, h1 = W.slice_group(w, b, g)
        if r1 == r0:
            continue
        q = W.bf16_bits_to_f64(qb[r0:r1, h0:h1])
        k = W.bf16_bits_to_f64(kb[r0:r1, g:g + 1])
        v = W.bf16_bits_to_f64(vb[r0:r1, g:g + 1])
        do = W.bf16_bits_to_f64(dob[r0:r1, h0:h1])
        cu = np.array([0, r1 - r0], dtype=np.int32)
        dq, dk, dv, o, lse = oracle.sdpa_bwd(q, k, v, do, cu, w.causal, w.scale)
        worst["o"] = max(worst["o"], float(np.max(np.abs(to_f64(gpu_out["o"][r0:r1, h0:h1]) - o))))
        worst["lse"] = max(worst["lse"], float(np.max(np.abs(to_f64(gpu_out["lse"][h0:h1, r0:r1]) - lse))))
        if "dq" in gpu_out:
            for name, ref, got in (("dq", dq, gpu_out["dq"][r0:r1, h0:h1]),
                                   ("dk", dk, gpu_out["dk"][r0:r1, g:g + 1]),
                                   ("dv", dv, gpu_out["dv"][r0:r1, g:g + 1])):
                # where the exact gradient vanishes (a single visible key) fall back to an absolute bound
                e = float(np.max(np.abs(to_f64(got) - ref)) / max(np.max(np.abs(ref)), GRAD_FLOOR))
                worst[name] = max(worst[name], e)
    return worst


def all_slices(w: W.Workload):
    return [(b, g) for b in range(w.B) for g in range(w.Hkv)]


def assert_within(worst, bwd=True):
    assert np.isfinite(worst["o"]) and worst["o"] <= TOL_O, worst
    assert np.isfinite(worst["lse"]) and worst["lse"] <= TOL_LSE, worst
    if bwd:
        for n in ("dq", "dk", "dv"):
            assert np.isfinite(worst[n]) and worst[n] <= TOL_GRAD, worst


def random_workload(lengths, Hq, Hkv, D, causal, seed, qk_mul=1.0):
    return W.Workload(f"t{seed}", seed, tuple(lengths), Hq, Hkv, D, causal, qk_mul)
