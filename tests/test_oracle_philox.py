"""The oracle's Philox4x32-10 against the published known-answer vectors, and the uniform map."""
import os

import numpy as np

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_kat.txt")


def test_philox_known_answers():
    n = 0
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        w = [int(x, 16) for x in line.split()]
        out = oracle.philox4x32_10(w[0:4], w[4:6])
        assert [int(x) for x in out] == w[6:10]
        n += 1
    assert n == 3


def test_uniform_is_word0_top24_bits_centred():
    seed, step = 0x0123456789ABCDEF, (5 << 32) | 17
    for (req, layer, purpose, index) in [(0, 1, 0, 0), (3, 2, 1, 0), (63, 9, 3, 7)]:
        ctr = [index, layer * 4 + purpose, req, step & 0xFFFFFFFF]
        key = [seed & 0xFFFFFFFF, (seed >> 32) ^ (step >> 32)]
        x0 = int(oracle.philox4x32_10(ctr, key)[0])
        u = oracle.uniform(seed, step, req, layer, purpose, index)
        assert u == ((x0 >> 8) + 0.5) / 2 ** 24
        assert 0.0 < u < 1.0 and float(np.float32(u)) == u   # exact in fp32 as well


def test_uniform_moments():
    u = np.array([oracle.uniform(11, 0, r, 1, 0, i) for r in range(200) for i in range(50)])
    assert abs(u.mean() - 0.5) < 0.01 and abs(u.var() - 1 / 12) < 0.005
    assert len(np.unique(u)) > 9990
