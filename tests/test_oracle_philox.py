"""Pins of the oracle's Philox4x32-10 and of the integer/float maps built on it."""
import os

import numpy as np

import oracle


def test_known_answer_vectors(golden_dir):
    rows = 0
    with open(os.path.join(golden_dir, "philox4x32_10_kat.txt")) as fh:
        for line in fh:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            w = [int(x, 16) for x in line.split()]
            assert oracle.philox4x32_10(w[0:4], w[4:6]) == w[6:10]
            rows += 1
    assert rows == 3


def test_bounded_is_floor_of_scaled_word():
    L = oracle.lib()
    rng = np.random.default_rng(0)
    for x in [0, 1, 2**31, 2**32 - 1] + [int(v) for v in rng.integers(0, 2**32, 200)]:
        for n in (1, 2, 3, 6, 64, 400):
            assert L.orc_bounded(x, n) == (x * n) // 2**32
    # the extremes map to the ends of the range
    assert L.orc_bounded(0, 64) == 0 and L.orc_bounded(2**32 - 1, 64) == 63


def test_uniform24_range_and_exactness():
    L = oracle.lib()
    assert L.orc_uniform24(0) == 0.0
    assert L.orc_uniform24(2**32 - 1) == (2**24 - 1) / 2**24 < 1.0
    assert L.orc_uniform24(0x80000000) == 0.5
    assert L.orc_uniform24(0x000000FF) == 0.0  # low 8 bits are dropped


def test_action_uniform_uses_word0_of_keyed_block():
    seed = 0x0123456789ABCDEF
    key = [seed & 0xFFFFFFFF, (seed >> 32) ^ 0x41435431]
    for t, e, a in [(0, 0, 0), (5, 17, 1), (1000, 32767, 7)]:
        word0 = oracle.philox4x32_10([t, e, a, 0], key)[0]
        assert oracle.lib().orc_action_uniform(seed, t, e, a) == (word0 >> 8) / 2**24
