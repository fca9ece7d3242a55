"""Python binding of the C ABI in include/sdpa.h: argument marshalling only.

Every step of the attention path runs in the CUDA library; torch supplies device memory and
streams.  There is no fallback: if the shared library is missing or cannot be loaded, or no
CUDA device is present, the calls raise.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("SDPA_B200_LIB", os.path.join(_HERE, "libsdpa_b200.so"))
_LIB = None

SDPA_OK = 0
EXPORTS = ("sdpa_fwd", "sdpa_bwd", "sdpa_bwd_workspace_bytes", "sdpa_query_status",
           "sdpa_status_string", "sdpa_last_cuda_error", "sdpa_host_staging_bytes",
           "sdpa_fwd_bwd_host", "sdpa_bwd_profile_events", "sdpa_bwd_static_scratch", "gemm_bf16_nt", "sdpa_selftest_wait_timeout", "sdpa_fwd_paged",
           "sdpa_fwd_bhsd", "sdpa_bwd_bhsd", "sdpa_bwd_deterministic", "sdpa_fwd_varlen_qk", "sdpa_bwd_varlen_qk",
           "sdpa_decode_paged", "sdpa_decode_paged_workspace_bytes")


class SdpaError(RuntimeError):
    pass


def load():
    """Load libsdpa_b200.so (built by paper_2608_17379_b200.build) and declare its signatures."""
    global _LIB
    if _LIB is not None:
        return _LIB
    if not os.path.exists(LIB_PATH):
        raise SdpaError(f"{LIB_PATH} is missing: run `python -m paper_2608_17379_b200.build` "
                        "(there is no CPU or library fallback)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, ci, cf = ctypes.c_void_p, ctypes.c_int, ctypes.c_float
    lib.sdpa_fwd.restype = ci
    lib.sdpa_fwd.argtypes = [vp, vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, cf, ci, ci, vp]
    lib.sdpa_bwd_workspace_bytes.restype = ctypes.c_size_t
    lib.sdpa_bwd_workspace_bytes.argtypes = [ci] * 6
    lib.sdpa_bwd.restype = ci
    lib.sdpa_bwd.argtypes = [vp] * 10 + [ci, ci, ci, ci, ci, cf, ci, ci, vp, ctypes.c_size_t, vp]
    lib.sdpa_fwd_varlen_qk.restype = ci
    lib.sdpa_fwd_varlen_qk.argtypes = [vp] * 7 + [ci, ci, ci, ci, ci, cf, ci, ci, ci, ci, vp]
    lib.sdpa_bwd_varlen_qk.restype = ci
    lib.sdpa_bwd_varlen_qk.argtypes = [vp] * 11 + [ci, ci, ci, ci, ci, cf, ci, ci, ci, ci, vp, ctypes.c_size_t, vp]
    lib.sdpa_decode_paged_workspace_bytes.restype = ctypes.c_size_t
    lib.sdpa_decode_paged_workspace_bytes.argtypes = [ci] * 5
    lib.sdpa_decode_paged.restype = ci
    lib.sdpa_decode_paged.argtypes = [vp] * 7 + [ci, ci, ci, ci, cf, ci, ci, vp, ctypes.c_size_t, vp]
    lib.sdpa_bwd_deterministic.restype = ci
    lib.sdpa_bwd_deterministic.argtypes = lib.sdpa_bwd.argtypes
    lib.sdpa_host_staging_bytes.restype = ctypes.c_size_t
    lib.sdpa_host_staging_bytes.argtypes = [ci] * 6
    lib.sdpa_fwd_bwd_host.restype = ci
    lib.sdpa_fwd_bwd_host.argtypes = [vp] * 10 + [ci, ci, ci, ci, ci, cf, ci, ci, vp, ctypes.c_size_t, vp]
    lib.sdpa_bwd_profile_events.restype = ci
    lib.sdpa_bwd_profile_events.argtypes = [vp, vp]
    lib.sdpa_bwd_static_scratch.restype = ci
    lib.sdpa_bwd_static_scratch.argtypes = [vp] * 10 + [ci, ci, ci, ci, ci, cf, ci, ci, vp]
    lib.sdpa_selftest_wait_timeout.restype = ci
    lib.sdpa_selftest_wait_timeout.argtypes = [ctypes.c_longlong, vp]
    lib.sdpa_fwd_paged.restype = ci
    lib.sdpa_fwd_paged.argtypes = [vp] * 8 + [ci, ci, ci, ci, ci, cf, ci, ci, ci, vp]
    lib.sdpa_fwd_bhsd.restype = ci
    lib.sdpa_fwd_bhsd.argtypes = [vp, vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, cf, vp]
    lib.sdpa_bwd_bhsd.restype = ci
    lib.sdpa_bwd_bhsd.argtypes = [vp] * 10 + [ci, ci, ci, ci, ci, ci, cf, vp, ctypes.c_size_t, vp]
    lib.gemm_bf16_nt.restype = ci
    lib.gemm_bf16_nt.argtypes = [vp, vp, vp, ci, ci, ci, vp]
    lib.sdpa_query_status.restype = ci
    lib.sdpa_query_status.argtypes = [vp, ctypes.POINTER(ci)]
    lib.sdpa_status_string.restype = ctypes.c_char_p
    lib.sdpa_status_string.argtypes = [ci]
    lib.sdpa_last_cuda_error.restype = ci
    lib.sdpa_last_cuda_error.argtypes = []
    _LIB = lib
    return lib


def status_string(code: int) -> str:
    return load().sdpa_status_string(int(code)).decode()


def _check(rc: int, what: str):
    if rc != SDPA_OK:
        lib = load()
        raise SdpaError(f"{what} failed: {rc} ({status_string(rc)}), cuda error {lib.sdpa_last_cuda_error()}")


def _stream_ptr(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream)


def _ptr(t) -> int:
    return 0 if t is None else int(t.data_ptr())


def _dims(q, k):
    assert q.dtype == torch.bfloat16 and k.dtype == torch.bfloat16
    assert q.is_contiguous() and k.is_contiguous() and q.dim() == 3 and k.dim() == 3
    T, Hq, D = q.shape
    return T, Hq, k.shape[1], D


def sdpa_fwd(q, k, v, cu_seqlens, max_seqlen: int, causal: bool, scale: float, o=None, lse=None, stream=None):
    """q [T,Hq,D], k,v [T,Hkv,D] bf16 CUDA tensors, cu_seqlens int32 [B+1] on the device.

    Returns (o bf16 [T,Hq,D], lse fp32 [Hq,T]); asynchronous on ``stream`` (default: current)."""
    lib = load()
    T, Hq, Hkv, D = _dims(q, k)
    B = cu_seqlens.numel() - 1
    assert cu_seqlens.dtype == torch.int32 and cu_seqlens.is_cuda
    if o is None:
        o = torch.empty_like(q)
    if lse is None:
        lse = torch.empty((Hq, T), dtype=torch.float32, device=q.device)
    rc = lib.sdpa_fwd(_ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse), _ptr(cu_seqlens), B, Hq, Hkv, D,
                      int(bool(causal)), float(scale), T, int(max_seqlen), _stream_ptr(stream))
    _check(rc, "sdpa_fwd")
    return o, lse


def sdpa_bwd_workspace_bytes(B, Hq, Hkv, D, total_tokens, max_seqlen) -> int:
    return int(load().sdpa_bwd_workspace_bytes(B, Hq, Hkv, D, total_tokens, max_seqlen))


def sdpa_bwd(q, k, v, o, lse, dout, cu_seqlens, max_seqlen: int, causal: bool, scale: float,
             dq=None, dk=None, dv=None, workspace=None, stream=None, deterministic: bool = False):
    """Gradients (dq, dk, dv) bf16 of sum(dout * O); o and lse are the outputs of sdpa_fwd.
    deterministic=True calls sdpa_bwd_deterministic (bit-reproducible dq)."""
    lib = load()
    T, Hq, Hkv, D = _dims(q, k)
    B = cu_seqlens.numel() - 1
    need = sdpa_bwd_workspace_bytes(B, Hq, Hkv, D, T, int(max_seqlen))
    if workspace is None:
        workspace = torch.empty(max(need, 256), dtype=torch.uint8, device=q.device)
    if dq is None:
        dq = torch.empty_like(q)
    if dk is None:
        dk = torch.empty_like(k)
    if dv is None:
        dv = torch.empty_like(v)
    fn = lib.sdpa_bwd_deterministic if deterministic else lib.sdpa_bwd
    rc = fn(_ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse), _ptr(dout), _ptr(dq), _ptr(dk), _ptr(dv),
            _ptr(cu_seqlens), B, Hq, Hkv, D, int(bool(causal)), float(scale), T, int(max_seqlen),
            _ptr(workspace), int(workspace.numel()), _stream_ptr(stream))
    _check(rc, "sdpa_bwd_deterministic" if deterministic else "sdpa_bwd")
    return dq, dk, dv


def sdpa_fwd_varlen_qk(q, k, v, cu_seqlens_q, cu_seqlens_k, max_seqlen_q: int, max_seqlen_k: int, causal: bool,
                       scale: float, o=None, lse=None, stream=None):
    """Separate key lengths: q [Tq,Hq,D], k,v [Tk,Hkv,D]; end-aligned causal mask.  Returns (o, lse [Hq,Tq])."""
    lib = load()
    Tq, Hq, Hkv, D = q.shape[0], q.shape[1], k.shape[1], q.shape[2]
    assert q.is_contiguous() and k.is_contiguous() and v.is_contiguous() and q.dtype == torch.bfloat16
    B = cu_seqlens_q.numel() - 1
    if o is None:
        o = torch.empty_like(q)
    if lse is None:
        lse = torch.empty((Hq, Tq), dtype=torch.float32, device=q.device)
    rc = lib.sdpa_fwd_varlen_qk(_ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse), _ptr(cu_seqlens_q), _ptr(cu_seqlens_k),
                                B, Hq, Hkv, D, int(bool(causal)), float(scale), Tq, k.shape[0], int(max_seqlen_q),
                                int(max_seqlen_k), _stream_ptr(stream))
    _check(rc, "sdpa_fwd_varlen_qk")
    return o, lse


def sdpa_bwd_varlen_qk(q, k, v, o, lse, dout, cu_seqlens_q, cu_seqlens_k, max_seqlen_q: int, max_seqlen_k: int,
                       causal: bool, scale: float, dq=None, dk=None, dv=None, workspace=None, stream=None):
    """Gradients for sdpa_fwd_varlen_qk."""
    lib = load()
    Tq, Hq, Hkv, D = q.shape[0], q.shape[1], k.shape[1], q.shape[2]
    B = cu_seqlens_q.numel() - 1
    need = sdpa_bwd_workspace_bytes(B, Hq, Hkv, D, Tq, int(max_seqlen_q))
    if workspace is None:
        workspace = torch.empty(max(need, 256), dtype=torch.uint8, device=q.device)
    dq = torch.empty_like(q) if dq is None else dq
    dk = torch.empty_like(k) if dk is None else dk
    dv = torch.empty_like(v) if dv is None else dv
    rc = lib.sdpa_bwd_varlen_qk(_ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse), _ptr(dout), _ptr(dq), _ptr(dk),
                                _ptr(dv), _ptr(cu_seqlens_q), _ptr(cu_seqlens_k), B, Hq, Hkv, D, int(bool(causal)),
                                float(scale), Tq, k.shape[0], int(max_seqlen_q), int(max_seqlen_k), _ptr(workspace),
                                int(workspace.numel()), _stream_ptr(stream))
    _check(rc, "sdpa_bwd_varlen_qk")
    return dq, dk, dv


def sdpa_decode_paged(q, k_cache, v_cache, kv_indptr, kv_indices, max_seqlen_k: int, scale: float, o=None,
                      lse=None, workspace=None, stream=None):
    """One query token per sequence over a page-size-1 cache: q [B,Hq,D], caches [P,Hkv,D].
    Returns (o [B,Hq,D] bf16, lse [Hq,B] fp32)."""
    lib = load()
    B, Hq, D = q.shape
    Hkv = k_cache.shape[1]
    assert q.is_contiguous() and k_cache.is_contiguous() and v_cache.is_contiguous() and q.dtype == torch.bfloat16
    need = int(lib.sdpa_decode_paged_workspace_bytes(B, Hq, Hkv, D, int(max_seqlen_k)))
    if workspace is None:
        workspace = torch.empty(max(need, 256), dtype=torch.uint8, device=q.device)
    if o is None:
        o = torch.empty_like(q)
    if lse is None:
        lse = torch.empty((Hq, B), dtype=torch.float32, device=q.device)
    rc = lib.sdpa_decode_paged(_ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(o), _ptr(lse), _ptr(kv_indptr),
                               _ptr(kv_indices), B, Hq, Hkv, D, float(scale), int(max_seqlen_k),
                               int(k_cache.shape[0]), _ptr(workspace), int(workspace.numel()), _stream_ptr(stream))
    _check(rc, "sdpa_decode_paged")
    return o, lse


def _dims_bhsd(q, k):
    assert q.dim() == 4 and k.dim() == 4 and q.is_contiguous() and k.is_contiguous()
    assert q.dtype == torch.bfloat16 and k.dtype == torch.bfloat16 and q.is_cuda and k.is_cuda
    B, Hq, S, D = q.shape
    assert k.shape[0] == B and k.shape[2] == S and k.shape[3] == D
    return B, Hq, k.shape[1], S, D


def sdpa_fwd_bhsd(q, k, v, causal: bool, scale: float, cu_seqlens=None, o=None, lse=None, stream=None):
    """Dense layout: q [B,Hq,S,D], k,v [B,Hkv,S,D] bf16 contiguous; cu_seqlens (optional int32 [B+1] on the
    device) gives per-sequence lengths <= S.  Returns (o [B,Hq,S,D] bf16, lse [B,Hq,S] fp32)."""
    lib = load()
    B, Hq, Hkv, S, D = _dims_bhsd(q, k)
    if o is None:
        o = torch.empty_like(q)
    if lse is None:
        lse = torch.empty((B, Hq, S), dtype=torch.float32, device=q.device)
    rc = lib.sdpa_fwd_bhsd(_ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse), _ptr(cu_seqlens) if cu_seqlens is not None else None,
                           B, Hq, Hkv, S, D, int(bool(causal)), float(scale), _stream_ptr(stream))
    _check(rc, "sdpa_fwd_bhsd")
    return o, lse


def sdpa_bwd_bhsd(q, k, v, o, lse, dout, causal: bool, scale: float, cu_seqlens=None, dq=None, dk=None, dv=None,
                  workspace=None, stream=None):
    """Gradients for the dense layout; tensors as in sdpa_fwd_bhsd."""
    lib = load()
    B, Hq, Hkv, S, D = _dims_bhsd(q, k)
    need = sdpa_bwd_workspace_bytes(B, Hq, Hkv, D, B * S, S)
    if workspace is None:
        workspace = torch.empty(max(need, 256), dtype=torch.uint8, device=q.device)
    dq = torch.empty_like(q) if dq is None else dq
    dk = torch.empty_like(k) if dk is None else dk
    dv = torch.empty_like(v) if dv is None else dv
    rc = lib.sdpa_bwd_bhsd(_ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse), _ptr(dout), _ptr(dq), _ptr(dk), _ptr(dv),
                           _ptr(cu_seqlens) if cu_seqlens is not None else None, B, Hq, Hkv, S, D,
                           int(bool(causal)), float(scale), _ptr(workspace), int(workspace.numel()),
                           _stream_ptr(stream))
    _check(rc, "sdpa_bwd_bhsd")
    return dq, dk, dv


STATIC_SCRATCH_BYTES = 32 << 20
SDPA_ERR_STATIC_SCRATCH = -7


def sdpa_bwd_static_scratch(q, k, v, o, lse, dout, cu_seqlens, max_seqlen: int, causal: bool, scale: float,
                            dq, dk, dv, stream=None):
    """sdpa_bwd without a workspace argument, for callers that must not allocate device memory:
    the scratch is a fixed 32 MiB array inside the library (see include/sdpa.h for the size limit,
    the first-call set-up and the rule that overlapping calls race on it).  The outputs dq, dk, dv
    are required, because this wrapper allocates nothing either.  Returns the library's return code
    instead of raising when the problem is too large for the built-in scratch."""
    lib = load()
    T, Hq, Hkv, D = _dims(q, k)
    B = cu_seqlens.numel() - 1
    rc = lib.sdpa_bwd_static_scratch(_ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse), _ptr(dout), _ptr(dq), _ptr(dk),
                                     _ptr(dv), _ptr(cu_seqlens), B, Hq, Hkv, D, int(bool(causal)), float(scale), T,
                                     int(max_seqlen), _stream_ptr(stream))
    if rc == SDPA_ERR_STATIC_SCRATCH:
        return rc
    _check(rc, "sdpa_bwd_static_scratch")
    return rc


def sdpa_host_staging_bytes(B, Hq, Hkv, D, total_tokens, max_seqlen) -> int:
    return int(load().sdpa_host_staging_bytes(B, Hq, Hkv, D, total_tokens, max_seqlen))


def sdpa_fwd_bwd_host(q, k, v, dout, o, lse, dq, dk, dv, cu_seqlens, max_seqlen: int, causal: bool, scale: float,
                      staging, stream=None):
    """Whole step on HOST tensors (pinned CPU torch tensors in, pinned CPU tensors out); ``staging``
    is a CUDA uint8 tensor of at least sdpa_host_staging_bytes(...) bytes.  Asynchronous."""
    lib = load()
    for t in (q, k, v, dout, o, lse, dq, dk, dv, cu_seqlens):
        assert not t.is_cuda and t.is_contiguous()
    assert staging.is_cuda
    T, Hq, Hkv, D = _dims(q, k)
    B = cu_seqlens.numel() - 1
    rc = lib.sdpa_fwd_bwd_host(_ptr(q), _ptr(k), _ptr(v), _ptr(dout), _ptr(o), _ptr(lse), _ptr(dq), _ptr(dk),
                               _ptr(dv), _ptr(cu_seqlens), B, Hq, Hkv, D, int(bool(causal)), float(scale), T,
                               int(max_seqlen), _ptr(staging), int(staging.numel()), _stream_ptr(stream))
    _check(rc, "sdpa_fwd_bwd_host")


def bwd_profile_events(start=None, stop=None):
    """Register two recorded-at-least-once torch.cuda.Event objects to be recorded around the main
    backward kernel by later sdpa_bwd calls of this thread (None, None switches it off)."""
    s = 0 if start is None else int(start.cuda_event)
    e = 0 if stop is None else int(stop.cuda_event)
    _check(load().sdpa_bwd_profile_events(s, e), "sdpa_bwd_profile_events")


def sdpa_fwd_paged(q, k_cache, v_cache, cu_seqlens_q, kv_indptr, kv_indices, max_seqlen_q: int, causal: bool,
                   scale: float, o=None, lse=None, stream=None):
    """Forward over a page-size-1 KV cache: q [Tq,Hq,D], k_cache/v_cache [num_pages,Hkv,D] bf16 CUDA
    tensors; cu_seqlens_q, kv_indptr int32 [B+1] and kv_indices int32 on the device."""
    lib = load()
    T, Hq, Hkv, D = _dims(q, k_cache)
    B = cu_seqlens_q.numel() - 1
    for t in (cu_seqlens_q, kv_indptr, kv_indices):
        assert t.dtype == torch.int32 and t.is_cuda
    if o is None:
        o = torch.empty_like(q)
    if lse is None:
        lse = torch.empty((Hq, T), dtype=torch.float32, device=q.device)
    rc = lib.sdpa_fwd_paged(_ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(o), _ptr(lse), _ptr(cu_seqlens_q),
                            _ptr(kv_indptr), _ptr(kv_indices), B, Hq, Hkv, D, int(bool(causal)), float(scale), T,
                            int(max_seqlen_q), int(k_cache.shape[0]), _stream_ptr(stream))
    _check(rc, "sdpa_fwd_paged")
    return o, lse


def gemm_bf16_nt(a, b, c=None, stream=None):
    """c [M,N] = a [M,K] @ b [N,K]^T, bf16 CUDA tensors, fp32 accumulation on the tensor cores."""
    lib = load()
    assert a.dtype == torch.bfloat16 and b.dtype == torch.bfloat16 and a.is_contiguous() and b.is_contiguous()
    M, K = a.shape
    N = b.shape[0]
    assert b.shape[1] == K
    if c is None:
        c = torch.empty((M, N), dtype=torch.bfloat16, device=a.device)
    _check(lib.gemm_bf16_nt(_ptr(a), _ptr(b), _ptr(c), M, N, K, _stream_ptr(stream)), "gemm_bf16_nt")
    return c


def query_status(stream=None):
    """Synchronise the stream and return (status, site) of the device status word (0 = fine)."""
    site = ctypes.c_int(0)
    rc = load().sdpa_query_status(_stream_ptr(stream), ctypes.byref(site))
    if rc < 0:
        _check(rc, "sdpa_query_status")
    return rc, site.value
