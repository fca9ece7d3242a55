"""Host-side checks that need no GPU: the shared library loads, exports every symbol the header
declares, and rejects bad arguments before touching CUDA."""
import ctypes
import os
import re

import pytest

from paper_2608_17379_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build_library()
    return binding.load()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "sdpa.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b((?:sdpa|gemm)_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert len(names) >= 6
    for n in names:
        assert hasattr(lib, n), n
    assert set(binding.EXPORTS) == set(names)


def test_status_strings(lib):
    assert binding.status_string(0) == "ok"
    for code in (-1, -2, -3, -4, -5, -6, 1, 2, 3):
        assert binding.status_string(code) not in ("ok", "unknown code")
    assert binding.status_string(99) == "unknown code"


def test_argument_checks_come_before_any_cuda_call(lib):
    buf = ctypes.create_string_buffer(4096)
    a = (ctypes.addressof(buf) + 255) & ~255
    fwd = lambda **kw: lib.sdpa_fwd(kw.get("q", a), a, a, a, a, kw.get("cu", a), kw.get("B", 1), kw.get("Hq", 2),
                                    kw.get("Hkv", 2), kw.get("D", 64), 0, kw.get("scale", 1.0), kw.get("T", 8),
                                    kw.get("L", 8), None)
    assert fwd(cu=None) == -1
    assert fwd(q=None) == -1
    assert fwd(q=a + 2) == -2
    assert fwd(D=100) == -3   # not a multiple of 8
    assert fwd(D=136) == -3   # above the largest kernel
    assert fwd(D=0) == -3
    assert fwd(Hq=3, Hkv=2) == -3
    assert fwd(B=0) == -3
    assert fwd(scale=0.0) == -3
    assert fwd(scale=float("nan")) == -3
    assert fwd(L=9, T=8) == -3
    assert fwd(T=0, L=0) == 0  # empty batch: valid no-op
    assert lib.sdpa_bwd_workspace_bytes(1, 2, 2, 100, 8, 8) == 0
    # head dimension 96 runs in the 128-wide kernel: the fp32 dQ accumulator is padded to 128 columns
    assert lib.sdpa_bwd_workspace_bytes(1, 2, 2, 96, 8, 8) == lib.sdpa_bwd_workspace_bytes(1, 2, 2, 128, 8, 8)
    need = lib.sdpa_bwd_workspace_bytes(1, 2, 2, 64, 8, 8)
    assert need >= 8 * 2 * 64 * 4 + 8 * 2 * 4
    bwd = lambda ws, n: lib.sdpa_bwd(a, a, a, a, a, a, a, a, a, a, 1, 2, 2, 64, 0, 1.0, 8, 8, ws, n, None)
    assert bwd(None, need) == -4
    assert bwd(a, need - 1) == -4
    assert bwd(a + 16, need) == -4
    assert lib.sdpa_host_staging_bytes(1, 2, 2, 64, 8, 8) > need
    det = lambda ws, n: lib.sdpa_bwd_deterministic(a, a, a, a, a, a, a, a, a, a, 1, 2, 2, 64, 0, 1.0, 8, 8, ws, n, None)
    assert det(None, need) == -4 and det(a, need - 1) == -4
    # dense [B, H, S, D] entry points: cu_seqlens is optional, the other checks are the same
    fd = lambda **kw: lib.sdpa_fwd_bhsd(kw.get("q", a), a, a, a, a, kw.get("cu", None), kw.get("B", 1), kw.get("Hq", 2),
                                        kw.get("Hkv", 2), kw.get("S", 8), kw.get("D", 64), 0, kw.get("scale", 1.0), None)
    assert fd(q=None) == -1
    assert fd(q=a + 2) == -2
    assert fd(D=100) == -3 and fd(Hq=3, Hkv=2) == -3 and fd(B=0) == -3 and fd(S=-1) == -3
    assert fd(B=1 << 20, S=1 << 20) == -3      # B * S must fit 32 bits
    assert fd(S=0) == 0                        # empty sequences: valid no-op
    bd = lambda ws, n: lib.sdpa_bwd_bhsd(a, a, a, a, a, a, a, a, a, None, 1, 2, 2, 8, 64, 0, 1.0, ws, n, None)
    assert bd(None, need) == -4 and bd(a, need - 1) == -4


def test_no_silent_fallback_without_a_gpu(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    buf = ctypes.create_string_buffer(4096)
    a = (ctypes.addressof(buf) + 255) & ~255
    rc = lib.sdpa_fwd(a, a, a, a, a, a, 1, 2, 2, 64, 0, 1.0, 8, 8, None)
    assert rc in (-5, -6)  # loud failure: no CUDA device / wrong architecture
