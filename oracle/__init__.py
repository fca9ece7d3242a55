"""fp64 CPU oracle for SDPA forward/backward (ctypes wrapper around sdpa_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the
bench's CPU-baseline / reference legs.  The product package never imports it
and it never imports the product package.

The C source is compiled with gcc on first use, on the machine it runs on
(-O3 -march=native -fopenmp, no fast-math), into ``oracle/build/``.
"""
from __future__ import annotations

import ctypes
import hashlib
import os
import platform
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sdpa_oracle.c")
_LIB = None


def _cpu_tag() -> str:
    flags = ""
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.startswith("flags"):
                    flags = line
                    break
    except OSError:
        pass
    return hashlib.sha1((platform.machine() + flags).encode()).hexdigest()[:8]


def build(force: bool = False) -> str:
    """Compile sdpa_oracle.c for this machine; return the path of the shared object."""
    with open(_SRC, "rb") as f:
        tag = hashlib.sha1(f.read()).hexdigest()[:10] + "_" + _cpu_tag()
    out_dir = os.path.join(_HERE, "build")
    os.makedirs(out_dir, exist_ok=True)
    so = os.path.join(out_dir, f"liboracle_{tag}.so")
    if force or not os.path.exists(so):
        tmp = so + f".tmp{os.getpid()}"
        cmd = ["gcc", "-O3", "-march=native", "-fopenmp", "-fPIC", "-shared", "-std=c11",
               "-o", tmp, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, so)
    return so


def _lib():
    global _LIB
    if _LIB is None:
        lib = ctypes.CDLL(build())
        dp = ctypes.POINTER(ctypes.c_double)
        ip = ctypes.POINTER(ctypes.c_int32)
        lib.oracle_sdpa_fwd.restype = ctypes.c_int
        lib.oracle_sdpa_fwd.argtypes = [dp, dp, dp, dp, dp, ip] + [ctypes.c_int] * 5 + [ctypes.c_double]
        lib.oracle_sdpa_bwd.restype = ctypes.c_int
        lib.oracle_sdpa_bwd.argtypes = [dp] * 9 + [ip] + [ctypes.c_int] * 5 + [ctypes.c_double]
        lib.oracle_num_threads.restype = ctypes.c_int
        _LIB = lib
    return _LIB


def num_threads() -> int:
    """Threads the oracle's OpenMP loops will use."""
    return int(_lib().oracle_num_threads())


def _f64(a, shape):
    a = np.ascontiguousarray(a, dtype=np.float64)
    assert a.shape == tuple(shape), (a.shape, shape)
    return a


def _p(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def sdpa_fwd(q, k, v, cu_seqlens, causal: bool, scale: float):
    """q [T,Hq,D], k,v [T,Hkv,D] float64 -> (o [T,Hq,D], lse [Hq,T]) float64."""
    q = np.ascontiguousarray(q, dtype=np.float64)
    T, Hq, D = q.shape
    Hkv = k.shape[1]
    k = _f64(k, (T, Hkv, D))
    v = _f64(v, (T, Hkv, D))
    cu = np.ascontiguousarray(cu_seqlens, dtype=np.int32)
    assert cu[0] == 0 and cu[-1] == T
    B = cu.shape[0] - 1
    o = np.zeros((T, Hq, D), dtype=np.float64)
    lse = np.zeros((Hq, T), dtype=np.float64)
    rc = _lib().oracle_sdpa_fwd(_p(q), _p(k), _p(v), _p(o), _p(lse),
                                cu.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)),
                                B, Hq, Hkv, D, int(bool(causal)), float(scale))
    if rc != 0:
        raise RuntimeError(f"oracle_sdpa_fwd failed: {rc}")
    return o, lse


def sdpa_bwd(q, k, v, dout, cu_seqlens, causal: bool, scale: float):
    """Gradients of sum(dout * O).  Returns (dq, dk, dv, o, lse), all float64."""
    q = np.ascontiguousarray(q, dtype=np.float64)
    T, Hq, D = q.shape
    Hkv = k.shape[1]
    k = _f64(k, (T, Hkv, D))
    v = _f64(v, (T, Hkv, D))
    dout = _f64(dout, (T, Hq, D))
    cu = np.ascontiguousarray(cu_seqlens, dtype=np.int32)
    assert cu[0] == 0 and cu[-1] == T
    B = cu.shape[0] - 1
    dq = np.zeros((T, Hq, D), dtype=np.float64)
    dk = np.zeros((T, Hkv, D), dtype=np.float64)
    dv = np.zeros((T, Hkv, D), dtype=np.float64)
    o = np.zeros((T, Hq, D), dtype=np.float64)
    lse = np.zeros((Hq, T), dtype=np.float64)
    rc = _lib().oracle_sdpa_bwd(_p(q), _p(k), _p(v), _p(dout), _p(dq), _p(dk), _p(dv), _p(o),
                                _p(lse), cu.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)),
                                B, Hq, Hkv, D, int(bool(causal)), float(scale))
    if rc != 0:
        raise RuntimeError(f"oracle_sdpa_bwd failed: {rc}")
    return dq, dk, dv, o, lse
