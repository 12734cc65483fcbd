"""Pins the oracle's counter-based generator to published known-answer vectors."""
import os

import numpy as np

GOLD = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_kat.txt")


def test_philox_known_answers(orc):
    n = 0
    for line in open(GOLD):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        w = [int(x, 16) for x in line.split()]
        assert orc.philox4x32_10(w[0:4], w[4:6]) == w[6:10]
        n += 1
    assert n == 3


def test_uniform_mapping(orc):
    # word 0 -> accept uniform, word 1 -> resample uniform, both (w >> 8) / 2^24 in [0, 1)
    seed, step, row, pos = 0x1234567890ABCDEF, 0x100000002, 7, 3
    w = orc.philox4x32_10([pos, row, step & 0xFFFFFFFF, step >> 32], [seed & 0xFFFFFFFF, seed >> 32])
    u, u2 = orc.review_uniforms(seed, step, row, pos)
    assert u == (w[0] >> 8) / 2.0 ** 24 and u2 == (w[1] >> 8) / 2.0 ** 24
    us = np.array([orc.review_uniforms(1, 0, r, 0) for r in range(4000)])
    assert us.min() >= 0.0 and us.max() < 1.0
    assert abs(us[:, 0].mean() - 0.5) < 0.03 and abs(us[:, 1].mean() - 0.5) < 0.03
    assert abs(np.corrcoef(us[:, 0], us[:, 1])[0, 1]) < 0.06
