"""Pins for the oracle's counter-based random numbers.

Philox4x32-10 itself is pinned by the known-answer vectors published with the generator's
reference implementation (tests/golden/philox4x32_10_kat.txt).  How counters are laid out and how
32 random bits become a uniform are this build's convention, stated here once more as a check on
the oracle's bookkeeping (the paper fixes no generator).
"""
import os

import numpy as np

import oracle

GOLD = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_kat.txt")


def test_known_answer_vectors():
    n = 0
    for line in open(GOLD):
        if line.startswith("#") or not line.strip():
            continue
        w = [int(x, 16) for x in line.split()]
        out = oracle.philox4x32_10(w[0:4], w[4:6])
        assert [int(x) for x in out] == w[6:10]
        n += 1
    assert n == 3


def test_counter_layout_and_uniform_mapping():
    seed = 0x1234_5678_9ABC_DEF0
    key = [seed & 0xFFFFFFFF, seed >> 32]
    # group G of 8 token ids: counter word 0 = ((G >> 10) << 8) | (G & 255), output word (G >> 8) & 3
    for step, row, G in [(0, 0, 0), (3, 17, 5), (15, 4095, 16_031), (1, 2, 300), (2, 9, 1023), (2, 9, 1024),
                         (7, 1, 70_000)]:
        ctr0 = ((G >> 10) << 8) | (G & 255)
        r = int(oracle.philox4x32_10([ctr0, step, row, 0], key)[(G >> 8) & 3])
        assert oracle.group_uniform(seed, step, row, G) == ((r >> 9) + 0.5) / 2 ** 23
        r = int(oracle.philox4x32_10([G, step, row, 3], key)[0])
        assert oracle.ingroup_uniform(seed, step, row, G) == ((r >> 9) + 0.5) / 2 ** 23
    # the layout is a bijection: no two groups share (counter, word)
    seen = {(((G >> 10) << 8) | (G & 255), (G >> 8) & 3) for G in range(20_000)}
    assert len(seen) == 20_000
    r = int(oracle.philox4x32_10([9, 0, 0, 1], key)[0])
    assert oracle.resample_uniform(seed, 9) == ((r >> 9) + 0.5) / 2 ** 23
    r = int(oracle.philox4x32_10([9, 2, 0, 2], key)[0])
    assert oracle.accept_uniform(seed, 9, 2) == ((r >> 9) + 0.5) / 2 ** 23


def test_uniforms_and_their_complements_are_fp32_exact_and_interior():
    u = np.array([oracle.group_uniform(5, 1, 2, G) for G in range(4000)])
    assert u.min() >= 2.0 ** -24 and u.max() <= 1 - 2.0 ** -24
    assert np.all(u.astype(np.float32).astype(np.float64) == u)
    assert np.all((1 - u).astype(np.float32).astype(np.float64) == 1 - u)
    # four groups sharing a counter get the four different output words
    assert len({oracle.group_uniform(5, 1, 2, G) for G in (7, 7 + 256, 7 + 512, 7 + 768)}) == 4
    # rough uniformity
    assert abs(u.mean() - 0.5) < 0.02 and abs((u < 0.25).mean() - 0.25) < 0.03
