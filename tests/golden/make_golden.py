"""Writes the stored expected values under tests/golden/.  It calls ONLY the float64 CPU oracle
(``oracle/``); nothing here comes from the CUDA library.  Run from the repository root:

    python tests/golden/make_golden.py

The paper prints no worked numerical example, so none of these values is the paper's.  What is stored:

* mask_mixed_P256_M32.txt   the retained bins of the synthetic per-layer masks (the stand-in for the
                            per-layer top-r*C chunks of the ablation study, Sec. 3.2) for a tiny grid;
                            integer-only, the generator is restated independently in the library.
* chunk_ranges_P2048_C22.txt  the C = 22 contiguous chunks of Sec. 3.2 / Eq. 6 on a grid of 2048 bins.
* greedy_keep_P64_C22.txt   greedy top-r*C selection (Sec. 3.2) from a fixed table of perplexity changes.
* iwdft_ramp_P8.txt         Eq. 4 on x[n] = n + 1, n < 4, zero-padded to P = 8, every one-sided bin; then
                            Eq. 9 / Eq. 12 (one more token, x[4] = -2); then Eq. 5 back (all bins: the input).
                            The same numbers follow by hand from the definition: C[k] = sum_n x[n] e^{-j pi k n / 4}.
"""
import os
import sys

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))
import oracle  # noqa: E402

SEED = 20030 * 1000 + 100 * 1          # seed rule of the synthetic workloads, configuration 1


def write(name, lines):
    with open(os.path.join(HERE, name), "w") as f:
        f.write("\n".join(lines) + "\n")


def main():
    oracle.build()
    # ---- masks
    lines = ["# P=256 M=32 seed=%d; one line per layer: layer, then the retained one-sided bins" % SEED]
    for layer in range(4):
        bins = oracle.plan(256, oracle.mask_mixed(256, 32, layer, SEED))
        lines.append("%d " % layer + " ".join(str(int(b)) for b in bins))
    write("mask_mixed_P256_M32.txt", lines)
    # ---- chunk ranges
    lines = ["# P=2048 C=22; chunk lo hi (two-sided bins [lo, hi))"]
    for c in range(22):
        lo, hi = oracle.chunk_range(2048, 22, c)
        lines.append("%d %d %d" % (c, lo, hi))
    write("chunk_ranges_P2048_C22.txt", lines)
    # ---- greedy selection
    delta = [((7 * c * c + 3 * c) % 23) / 8.0 for c in range(22)]      # has ties
    lines = ["# P=64 C=22 delta[c]=((7c^2+3c) mod 23)/8; ratio, n_keep, then the kept one-sided bins"]
    for ratio in (0.05, 0.125, 0.25, 0.5):
        mask, n_keep = oracle.mask_from_scores(64, 22, delta, ratio)
        lines.append("%g %d " % (ratio, n_keep) + " ".join(str(int(k)) for k in np.nonzero(mask)[0]))
    write("greedy_keep_P64_C22.txt", lines)
    # ---- a tiny transform, update and reconstruction
    P = 8
    bins = oracle.plan(P, np.ones(P // 2 + 1, dtype=np.uint8))
    x = np.array([[1.0], [2.0], [3.0], [4.0]])
    re, im = oracle.compress(x, P, bins)
    re, im = np.ascontiguousarray(re), np.ascontiguousarray(im)
    lines = ["# P=8, x = 1 2 3 4, bins 0..4: Re C[k], Im C[k] (Eq. 4)"]
    lines += ["%d %.17g %.17g" % (k, re[i, 0], im[i, 0]) for i, k in enumerate(bins)]
    oracle.append(re, im, P, bins, 4, np.array([-2.0]))
    lines.append("# after the update with x[4] = -2 at position 4 (Eq. 9 / Eq. 12)")
    lines += ["%d %.17g %.17g" % (k, re[i, 0], im[i, 0]) for i, k in enumerate(bins)]
    rec = oracle.reconstruct(re, im, P, bins, 5)
    lines.append("# reconstruction of the first 5 positions (Eq. 5)")
    lines += ["%d %.17g" % (n, rec[n, 0]) for n in range(5)]
    write("iwdft_ramp_P8.txt", lines)


if __name__ == "__main__":
    main()
