"""Writes tests/golden/config1_oracle.txt: sampled fp64 outputs of the CPU oracle on the
single-linear configuration (seed 0, 2048x2048, keep rates 1.0 and 0.85).  Calls only
oracle/ and the seeded input generators; re-run it if the generators change.

    python tests/golden/make_golden.py
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import oracle  # noqa: E402
from paper_2512_03383_b200 import synth  # noqa: E402


def config1(seed=0):
    rng = np.random.default_rng(seed)
    qw = synth.draw_qweight(rng, 2048, 2048, std=0.02)
    x = synth.draw_x(rng, 1, 2048, "f16")
    return qw, x


SAMPLES = [0, 1, 2, 127, 128, 129, 511, 1000, 1023, 1024, 1500, 1738, 1739]


def compute():
    qw, x = config1()
    packed = oracle.pack_u4(qw.codes)
    lines = []
    for rate in (1.0, 0.85):
        k = synth.keep_count(rate, 2048)
        acc = oracle.qlinear(x[:, :k], packed, qw.scales, qw.zeros, oracle.leading(k), oracle.leading(k))
        for j in SAMPLES:
            lines.append("%.2f %d %d %s" % (rate, k, j, float(acc[0, j]).hex()))
    return lines


if __name__ == "__main__":
    out = os.path.join(os.path.dirname(os.path.abspath(__file__)), "config1_oracle.txt")
    with open(out, "w") as f:
        f.write("# keep_rate k output_index fp64(hex) -- written by make_golden.py from oracle/ only\n")
        f.write("\n".join(compute()) + "\n")
    print("wrote", out)
