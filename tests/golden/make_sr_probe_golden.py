"""Writes tests/golden/sr_e2m1x4_probe.txt from the raw record of a hardware probe.

The probe ran once on a B200: a kernel fed `cvt.rs.satfinite.e2m1x4.f32` (sm_100a's
stochastic-rounding conversion of four FP32 values with one 32-bit random word) with
1 540 672 inputs and stored what came back.  Record layout (little endian): uint64 n, uint64
n_structured, then n x 4 float32 inputs, n uint32 random words, n uint32 results (four nibbles,
element 0 in bits 3:0).  The first n_structured records walk single values through every grid
interval in steps of 1/256 of the interval with all-zero, all-one, single-bit and
all-but-one-bit random words; the rest are uniform random values in (-7, 7) with random words.

This script takes nothing from any library: it samples records from the file it is given
(every k-th structured and every k-th random one, fixed strides) and prints them as text, one
record per line: the bit patterns of the four inputs, the random word and the result, in hex.
The oracle's stochastic-rounding rule is replayed on these lines by tests/test_oracle_momentum.py.

    python tests/golden/make_sr_probe_golden.py <probe.bin> > tests/golden/sr_e2m1x4_probe.txt
"""
import sys

import numpy as np


def main():
    with open(sys.argv[1], "rb") as f:
        n, ns = (int(v) for v in np.frombuffer(f.read(16), np.uint64))
        y = np.frombuffer(f.read(16 * n), np.uint32).reshape(n, 4)
        word = np.frombuffer(f.read(4 * n), np.uint32)
        out = np.frombuffer(f.read(4 * n), np.uint32)
    picks = list(range(0, ns, ns // 400)) + list(range(ns, n, (n - ns) // 400))
    print("# cvt.rs.satfinite.e2m1x4.f32 on sm_100a, recorded on a B200: y0 y1 y2 y3 (FP32 bit patterns), random word, result")
    print(f"# {len(picks)} of {n} records ({ns} structured, the rest random)")
    for i in picks:
        print(" ".join(f"{int(v):08x}" for v in y[i]), f"{int(word[i]):08x}", f"{int(out[i]) & 0xFFFF:04x}")


if __name__ == "__main__":
    main()
