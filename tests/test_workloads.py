"""The seeded input generator: reproducible, sliceable, right distributions."""
import os

import numpy as np

import oracle
from paper_2608_17379_b200 import workloads as W

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def test_stream_matches_stored_values():
    lines = [l.split() for l in open(os.path.join(GOLD, "generator_stream.txt")) if not l.startswith("#")]
    for tid, line in zip((W.TENSOR_Q, W.TENSOR_K, W.TENSOR_V, W.TENSOR_DO), lines[:4]):
        bits = W.gen_tensor_bits(0, tid, (16,))
        assert [f"{int(b):04x}" for b in bits] == line
    assert [str(int(x)) for x in W.gen_lengths(4, 8, 512, 8192)] == lines[4]


def test_normal_moments():
    z = W.normal_f64(7, W.TENSOR_Q, 0, 1_000_000)
    assert abs(z.mean()) < 5e-3 and abs(z.var() - 1.0) < 5e-3
    assert abs(((z - z.mean()) ** 4).mean() / z.var() ** 2 - 3.0) < 0.05
    assert np.all(np.isfinite(z))


def test_slices_reproduce_the_whole():
    full = W.gen_tensor_bits(3, W.TENSOR_K, (50, 4, 8))
    part = W.gen_tensor_bits(3, W.TENSOR_K, (10, 4, 8), start=20 * 32)
    assert np.array_equal(full[20:30], part)
    assert not np.array_equal(W.gen_tensor_bits(4, W.TENSOR_K, (10,)), W.gen_tensor_bits(3, W.TENSOR_K, (10,)))
    assert not np.array_equal(W.gen_tensor_bits(3, W.TENSOR_V, (10,)), W.gen_tensor_bits(3, W.TENSOR_K, (10,)))


def test_bf16_rounding_is_nearest_even_and_mul2_is_exact_doubling():
    x = np.array([1.0, 1.00390625, 1.01171875, -1.00390625, 3.0e-3], dtype=np.float32)
    # 1 + 2^-8 is a tie between 1.0 and 1+2^-7 -> even (1.0); 1 + 3*2^-8 ties to 1+2^-6
    got = W.bf16_bits_to_f64(W.f32_to_bf16_bits(x))
    assert got[0] == 1.0 and got[1] == 1.0 and got[2] == 1.015625 and got[3] == -1.0
    assert abs(got[4] - 3.0e-3) <= 3.0e-3 * 2 ** -8
    a = W.bf16_bits_to_f64(W.gen_tensor_bits(5, W.TENSOR_Q, (4096,), 1.0))
    b = W.bf16_bits_to_f64(W.gen_tensor_bits(5, W.TENSOR_Q, (4096,), 2.0))
    assert np.array_equal(2.0 * a, b)


def test_lengths_and_configs():
    lens = W.gen_lengths(4, 8, 512, 8192)
    assert lens.min() >= 512 and lens.max() <= 8192
    assert any(int(l) % 128 for l in lens)
    many = W.gen_lengths(9, 20000, 512, 8192)
    assert 512 <= many.min() < 520 and 8184 < many.max() <= 8192
    c3 = W.config("c3")
    assert (c3.B, c3.T, c3.Hq, c3.Hkv, c3.D, c3.causal) == (2, 8192, 32, 8, 128, True)
    assert abs(c3.fwd_flops() - 274.9e9) < 0.1e9 and abs(c3.bwd_flops() - 687.2e9) < 0.1e9
    c5 = W.config("c5")
    assert c5.B == 8 and c5.cu_seqlens[-1] == c5.T and c5.Hq // c5.Hkv == 8
    assert W.config("c4").qk_mul == 2.0 and not W.config("c4").causal and W.config("c4c").causal


def test_oracle_c1_matches_stored_samples():
    w = W.config("c1")
    q, k, v, do = (W.bf16_bits_to_f64(x) for x in W.make_inputs(w))
    dq, dk, dv, o, lse = oracle.sdpa_bwd(q, k, v, do, w.cu_seqlens, w.causal, w.scale)
    t = {"o": o, "lse": lse, "dq": dq, "dk": dk, "dv": dv}
    for line in open(os.path.join(GOLD, "oracle_c1_samples.txt")):
        if line.startswith("#"):
            continue
        name, idx, val = line.split()
        assert abs(t[name].reshape(-1)[int(idx)] - float(val)) < 1e-12
