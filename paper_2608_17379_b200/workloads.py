"""Seeded synthetic inputs for the bf16 SDPA forward/backward path.

This module only produces inputs (tensor values, sequence lengths, workload
shapes).  It contains none of the attention arithmetic, so the CPU oracle and
the CUDA path can both be fed from it without sharing any of the method.

The paper measures on fixed attention workloads (App. "Workloads": bf16,
batch 4, 48 heads, sequence 4096, head dim 128; and a ragged GQA prefill with
32 query / 4 KV heads over 33 packed sequences).  Those records are not
available here, so the five configurations below take their shapes and value
distributions and stand in for them.

Every value is a pure function of (seed, tensor id, flat element index): a
counter-based generator.  Any slice of any tensor can therefore be produced on
its own, which is what lets the slow oracle check one (sequence, kv-group)
slice of a large configuration.

bf16 values travel as ``numpy.uint16`` bit patterns (numpy has no bf16 type).
"""
from __future__ import annotations

import dataclasses
import math

import numpy as np

TENSOR_Q, TENSOR_K, TENSOR_V, TENSOR_DO, TENSOR_LENGTHS = 1, 2, 3, 4, 5

_M64 = np.uint64(0xFFFFFFFFFFFFFFFF)
_GAMMA = np.uint64(0x9E3779B97F4A7C15)
_C1 = np.uint64(0xBF58476D1CE4E5B9)
_C2 = np.uint64(0x94D049BB133111EB)


def _mix64(x: np.ndarray) -> np.ndarray:
    """splitmix64 finaliser on a uint64 array (wrapping arithmetic)."""
    with np.errstate(over="ignore"):
        z = x + _GAMMA
        z = (z ^ (z >> np.uint64(30))) * _C1
        z = (z ^ (z >> np.uint64(27))) * _C2
        return z ^ (z >> np.uint64(31))


def _stream_key(seed: int, tensor_id: int) -> np.uint64:
    k = _mix64(np.array([(seed * 0x100 + tensor_id) & 0xFFFFFFFFFFFFFFFF], dtype=np.uint64))
    return _mix64(k)[0]


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit pattern, round to nearest even (finite inputs)."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = b + np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1))
    return (r >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """bf16 bit pattern -> float64 (exact)."""
    w = np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return w.view(np.float32).astype(np.float64)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    w = np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return w.view(np.float32)


def normal_f64(seed: int, tensor_id: int, start: int, count: int) -> np.ndarray:
    """Standard normal samples for flat indices [start, start+count) (Box-Muller)."""
    key = _stream_key(seed, tensor_id)
    out = np.empty(count, dtype=np.float64)
    chunk = 1 << 22
    two53 = 1.0 / 9007199254740992.0
    for off in range(0, count, chunk):
        n = min(chunk, count - off)
        idx = np.arange(start + off, start + off + n, dtype=np.uint64)
        with np.errstate(over="ignore"):
            h1 = _mix64(key ^ (idx * np.uint64(2)))
            h2 = _mix64(key ^ (idx * np.uint64(2) + np.uint64(1)))
        u1 = ((h1 >> np.uint64(11)).astype(np.float64) + 1.0) * two53  # (0, 1]
        u2 = (h2 >> np.uint64(11)).astype(np.float64) * two53  # [0, 1)
        out[off:off + n] = np.sqrt(-2.0 * np.log(u1)) * np.cos((2.0 * math.pi) * u2)
    return out


def gen_tensor_bits(seed: int, tensor_id: int, shape, mul: float = 1.0,
                    start: int = 0) -> np.ndarray:
    """bf16 bit patterns of ``mul * N(0,1)`` for a contiguous tensor of ``shape``.

    ``start`` is the flat index of the first element inside the (larger) tensor
    the values belong to, so that slices reproduce the values of the whole.
    """
    count = int(np.prod(shape))
    z = normal_f64(seed, tensor_id, start, count) * float(mul)
    return f32_to_bf16_bits(z.astype(np.float32)).reshape(shape)


def gen_lengths(seed: int, n: int, lo: int, hi: int) -> np.ndarray:
    """``n`` integers uniform on [lo, hi] inclusive, from the seed."""
    key = _stream_key(seed, TENSOR_LENGTHS)
    h = _mix64(key ^ np.arange(n, dtype=np.uint64))
    return (lo + (h % np.uint64(hi - lo + 1))).astype(np.int64)


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    seed: int
    lengths: tuple  # per-sequence token counts
    Hq: int
    Hkv: int
    D: int
    causal: bool
    qk_mul: float = 1.0

    @property
    def B(self) -> int:
        return len(self.lengths)

    @property
    def T(self) -> int:
        return int(sum(self.lengths))

    @property
    def max_seqlen(self) -> int:
        return int(max(self.lengths)) if self.lengths else 0

    @property
    def scale(self) -> float:
        return 1.0 / math.sqrt(self.D)

    @property
    def cu_seqlens(self) -> np.ndarray:
        cu = np.zeros(self.B + 1, dtype=np.int32)
        cu[1:] = np.cumsum(np.asarray(self.lengths, dtype=np.int64))
        return cu

    def fwd_flops(self) -> float:
        s = float(sum(int(l) * int(l) for l in self.lengths))
        f = 4.0 * self.Hq * self.D * s
        return f * 0.5 if self.causal else f

    def bwd_flops(self) -> float:
        return 2.5 * self.fwd_flops()

    def min_bytes_fwd(self) -> float:
        return self.T * (2 * self.Hq * self.D * 2 + 2 * self.Hkv * self.D * 2 + 4 * self.Hq)

    def min_bytes_bwd(self) -> float:
        return self.T * (4 * self.Hq * self.D * 2 + 4 * self.Hkv * self.D * 2 + 4 * self.Hq)


def config(name: str) -> Workload:
    """The five benchmark configurations (c1..c5; c4 has a causal and a full variant)."""
    if name == "c1":
        return Workload("c1", 0, (128,), 2, 2, 64, False)
    if name == "c2":
        return Workload("c2", 1, (2048,) * 4, 16, 16, 128, True)
    if name == "c3":
        return Workload("c3", 2, (4096,) * 2, 32, 8, 128, True)
    if name == "c4":
        return Workload("c4", 3, (16384,), 16, 16, 128, False, qk_mul=2.0)
    if name == "c4c":
        return Workload("c4c", 3, (16384,), 16, 16, 128, True, qk_mul=2.0)
    if name == "c5":
        lens = tuple(int(x) for x in gen_lengths(4, 8, 512, 8192))
        return Workload("c5", 4, lens, 32, 4, 128, True)
    # The paper's own primary attention shape (appendix "Workloads": batch 4, 48 heads, sequence 4096)
    # and its d64 / d96 generalisation shapes; context workloads, not part of the five benchmark configs.
    if name == "mha":
        return Workload("mha", 5, (4096,) * 4, 48, 48, 128, False)
    if name == "mha_causal":
        return Workload("mha_causal", 5, (4096,) * 4, 48, 48, 128, True)
    if name == "mha_d64":
        return Workload("mha_d64", 6, (4096,) * 4, 48, 48, 64, True)
    if name == "mha_d96":
        return Workload("mha_d96", 7, (4096,) * 4, 48, 48, 96, True)
    raise KeyError(name)


CONFIG_NAMES = ("c1", "c2", "c3", "c4", "c4c", "c5", "mha", "mha_causal", "mha_d64", "mha_d96")


def make_inputs(w: Workload):
    """Full q, k, v, do tensors of a workload as bf16 bit patterns, token-major [T, H, D]."""
    q = gen_tensor_bits(w.seed, TENSOR_Q, (w.T, w.Hq, w.D), w.qk_mul)
    k = gen_tensor_bits(w.seed, TENSOR_K, (w.T, w.Hkv, w.D), w.qk_mul)
    v = gen_tensor_bits(w.seed, TENSOR_V, (w.T, w.Hkv, w.D), 1.0)
    do = gen_tensor_bits(w.seed, TENSOR_DO, (w.T, w.Hq, w.D), 1.0)
    return q, k, v, do


def slice_group(w: Workload, b: int, g: int):
    """Index helpers for the independent (sequence b, kv head g) slice of a workload.

    Returns (row0, row1, h0, h1): token rows [row0,row1) and query heads [h0,h1).
    """
    cu = w.cu_seqlens
    G = w.Hq // w.Hkv
    return int(cu[b]), int(cu[b + 1]), g * G, (g + 1) * G
