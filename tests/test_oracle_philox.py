"""Pins for the oracle's Philox4x32-10 and its uniform conversion."""
import os

import numpy as np

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_kat.txt")


def test_known_answer_vectors():
    n = 0
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        w = [int(x, 16) for x in line.split()]
        out = oracle.philox4x32_10(w[0:4], w[4:6])
        assert [int(x) for x in out] == w[6:10], line
        n += 1
    assert n == 3


def test_counter_words_are_distinguished():
    base = oracle.philox4x32_10([5, 6, 7, 0], [11, 12])
    seen = {tuple(int(x) for x in base)}
    # changing any single counter or key word changes the block
    for j in range(4):
        c = [5, 6, 7, 0]
        c[j] += 1
        seen.add(tuple(int(x) for x in oracle.philox4x32_10(c, [11, 12])))
    for j in range(2):
        k = [11, 12]
        k[j] += 1
        seen.add(tuple(int(x) for x in oracle.philox4x32_10([5, 6, 7, 0], k)))
    assert len(seen) == 7


def test_uniform24_range_and_grid():
    assert oracle.uniform24(0) == 0.0
    assert oracle.uniform24(0xFF) == 0.0
    assert oracle.uniform24(0x100) == 2.0 ** -24
    assert oracle.uniform24(0xFFFFFFFF) == 1.0 - 2.0 ** -24


def test_uniformity_chi_square():
    # 2^16 consecutive counters, word 0 -> 64 equal bins
    n = 1 << 16
    u = np.empty(n)
    for i in range(n):
        u[i] = oracle.uniform24(int(oracle.philox4x32_10([i, 0, 0, 0], [123, 456])[0]))
    hist, _ = np.histogram(u, bins=64, range=(0.0, 1.0))
    exp = n / 64
    chi2 = float(((hist - exp) ** 2 / exp).sum())
    # 63 degrees of freedom: mean 63, std ~11.2; 130 is > 5 sigma
    assert chi2 < 130.0, chi2
    assert abs(u.mean() - 0.5) < 5 * (1 / np.sqrt(12 * n))
