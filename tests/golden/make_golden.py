"""Writes the stored expected values under tests/golden/.

Calls only the seeded input generator and the CPU oracle (never the CUDA path).
The paper prints no numeric example of an attention output, so these files pin
nothing about the method itself; they freeze the generator's stream and the
oracle's c1 outputs so that an accidental change to either is caught.

Run from the repository root:  python tests/golden/make_golden.py
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import oracle  # noqa: E402
from paper_2608_17379_b200 import workloads as W  # noqa: E402

HERE = os.path.dirname(os.path.abspath(__file__))


def main():
    with open(os.path.join(HERE, "generator_stream.txt"), "w") as f:
        f.write("# bf16 bit patterns (hex) of the first 16 elements, seed 0, tensors Q K V dO; then c5 lengths\n")
        for tid in (W.TENSOR_Q, W.TENSOR_K, W.TENSOR_V, W.TENSOR_DO):
            bits = W.gen_tensor_bits(0, tid, (16,))
            f.write(" ".join(f"{int(b):04x}" for b in bits) + "\n")
        f.write(" ".join(str(int(x)) for x in W.gen_lengths(4, 8, 512, 8192)) + "\n")
    w = W.config("c1")
    q, k, v, do = (W.bf16_bits_to_f64(x) for x in W.make_inputs(w))
    dq, dk, dv, o, lse = oracle.sdpa_bwd(q, k, v, do, w.cu_seqlens, w.causal, w.scale)
    with open(os.path.join(HERE, "oracle_c1_samples.txt"), "w") as f:
        f.write("# oracle outputs on config c1 (seed 0): tensor index value (repr of float64)\n")
        rng = np.random.default_rng(123)
        for name, x in (("o", o), ("lse", lse), ("dq", dq), ("dk", dk), ("dv", dv)):
            flat = x.reshape(-1)
            for i in rng.choice(flat.size, 6, replace=False):
                f.write(f"{name} {int(i)} {float(flat[i])!r}\n")


if __name__ == "__main__":
    main()
