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


def _philox4x32_10_plain(ctr, key):
    """Philox4x32-10 written out from its published definition (Salmon et al., SC'11) with Python integers:
    ten rounds of two 32x32 -> 64-bit multiplications, the high halves xor-ed with the other counter words
    and the round key; the key grows by the Weyl constants between rounds."""
    M0, M1, W0, W1, MASK = 0xD2511F53, 0xCD9E8D57, 0x9E3779B9, 0xBB67AE85, 0xFFFFFFFF
    c0, c1, c2, c3 = (int(x) & MASK for x in ctr)
    k0, k1 = (int(x) & MASK for x in key)
    for _ in range(10):
        p0, p1 = M0 * c0, M1 * c2
        c0, c1, c2, c3 = ((p1 >> 32) ^ c1 ^ k0) & MASK, p1 & MASK, ((p0 >> 32) ^ c3 ^ k1) & MASK, p0 & MASK
        k0, k1 = (k0 + W0) & MASK, (k1 + W1) & MASK
    return [c0, c1, c2, c3]


def test_second_implementation_agrees_on_random_counters():
    # the plain-integer version reproduces the published vectors itself ...
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        w = [int(x, 16) for x in line.split()]
        assert _philox4x32_10_plain(w[0:4], w[4:6]) == w[6:10]
    # ... and agrees with the oracle's on counters and keys of every size
    rng = np.random.default_rng(2024)
    for _ in range(2000):
        ctr = [int(x) for x in rng.integers(0, 1 << 32, size=4, dtype=np.uint64)]
        key = [int(x) for x in rng.integers(0, 1 << 32, size=2, dtype=np.uint64)]
        assert [int(x) for x in oracle.philox4x32_10(ctr, key)] == _philox4x32_10_plain(ctr, key)
    # the counter layout of the step: (position, sequence, iteration, purpose), small integers
    for pos in (0, 1, 575, 2303):
        for seq in (0, 15):
            for it in (0, 7):
                for purpose in range(6):
                    ctr = [pos, seq, it, purpose]
                    assert [int(x) for x in oracle.philox4x32_10(ctr, [7, 0])] == _philox4x32_10_plain(ctr, [7, 0])


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
