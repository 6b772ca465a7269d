"""Stored expected values (tests/golden/, written by tests/golden/make_golden.py from the oracle alone)
against (a) the oracle as it stands, (b) the definition evaluated by hand in this file, and (c) the
library's host-side integer logic.  No GPU needed."""
import cmath
import os

import numpy as np
import pytest

GOLD = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
SEED = 20030 * 1000 + 100 * 1


def _rows(name):
    with open(os.path.join(GOLD, name)) as f:
        return [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]


@pytest.fixture(scope="module")
def lib():
    from paper_2507_20030_b200 import binding, build
    build.build()
    binding.load()
    return binding


def test_mask_golden_oracle_and_library(oracle, lib):
    rows = _rows("mask_mixed_P256_M32.txt")
    assert len(rows) == 4
    for r in rows:
        layer, bins = int(r[0]), np.array(r[1:], dtype=np.int32)
        assert bins.shape == (32,) and np.all(np.diff(bins) > 0)
        assert np.array_equal(oracle.plan(256, oracle.mask_mixed(256, 32, layer, SEED)), bins)
        assert np.array_equal(np.nonzero(lib.mask_mixed(256, 32, layer, SEED))[0], bins)
    assert len({tuple(r[1:]) for r in rows}) > 1            # the layers differ


def test_chunk_ranges_golden(oracle, lib):
    rows = _rows("chunk_ranges_P2048_C22.txt")
    assert len(rows) == 22
    for c, lo, hi in ((int(a), int(b), int(d)) for a, b, d in rows):
        assert oracle.chunk_range(2048, 22, c) == (lo, hi) == tuple(lib.chunk_range(2048, 22, c))
    # Sec. 3.2: contiguous chunks of floor(P / C) bins that tile the grid, the last one taking the remainder
    assert rows[0][1] == "0" and rows[-1][2] == "2048"
    assert all(int(r[2]) - int(r[1]) == 2048 // 22 for r in rows[:-1])


def test_greedy_selection_golden(oracle, lib):
    delta = [((7 * c * c + 3 * c) % 23) / 8.0 for c in range(22)]
    for r in _rows("greedy_keep_P64_C22.txt"):
        ratio, n_keep, bins = float(r[0]), int(r[1]), np.array(r[2:], dtype=np.int64)
        assert n_keep == max(1, int(np.floor(ratio * 22 + 0.5)))         # reading of "r * C chunks"
        for impl in (oracle, lib):
            mask, n = impl.mask_from_scores(64, 22, delta, ratio)
            assert n == n_keep and np.array_equal(np.nonzero(mask)[0], bins)


def test_iwdft_ramp_golden_against_the_definition(oracle):
    rows = _rows("iwdft_ramp_P8.txt")
    first, second, rec = rows[:5], rows[5:10], rows[10:]
    P = 8
    x = [1.0, 2.0, 3.0, 4.0]
    for r in first:                                          # Eq. 4 by hand
        k = int(r[0])
        want = sum(x[n] * cmath.exp(-2j * cmath.pi * k * n / P) for n in range(4))
        assert abs(complex(float(r[1]), float(r[2])) - want) < 1e-14
    for r in second:                                         # Eq. 9 / Eq. 12: one more token at position 4
        k = int(r[0])
        want = sum(x[n] * cmath.exp(-2j * cmath.pi * k * n / P) for n in range(4)) - 2.0 * cmath.exp(-2j * cmath.pi * k * 4 / P)
        assert abs(complex(float(r[1]), float(r[2])) - want) < 1e-14
    assert np.allclose([float(r[1]) for r in rec], [1, 2, 3, 4, -2], atol=1e-14)      # Eq. 5, every bin kept
    # and the oracle as it stands reproduces the file
    bins = oracle.plan(P, np.ones(P // 2 + 1, dtype=np.uint8))
    re, im = oracle.compress(np.array(x)[:, None], P, bins)
    assert np.allclose(re[:, 0], [float(r[1]) for r in first], atol=1e-15)
    assert np.allclose(im[:, 0], [float(r[2]) for r in first], atol=1e-15)
