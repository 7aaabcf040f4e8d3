"""Pins for the oracle's Philox4x32-10 and its slot addressing."""
import os

import numpy as np

from oracle import philox

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_kat.txt")


def _vectors():
    for line in open(GOLDEN):
        line = line.split("#")[0].strip()
        if not line:
            continue
        w = [int(x, 16) for x in line.split()]
        yield w[0:4], w[4:6], tuple(w[6:10])


def test_known_answer_vectors():
    vs = list(_vectors())
    assert len(vs) == 3
    for ctr, key, out in vs:
        assert philox.philox4x32_10(ctr, key) == out


def test_against_numpy_philox_structure():
    """numpy ships the 64-bit-word Philox4x64; it cannot check our words, but our generator must
    at least be a bijection of the counter for a fixed key (a round function that dropped a word
    would collide)."""
    seen = set()
    for c0 in range(64):
        for c1 in range(64):
            seen.add(philox.philox4x32_10((c0, c1, 0, 0), (1, 2)))
    assert len(seen) == 64 * 64


def test_u24_range_and_slots():
    seed, step = 0x1234_5678_9ABC_DEF0, (1 << 33) + 5
    vals = [philox.u24(seed, step, 3, s) for s in range(24)]
    assert all(0 <= v < (1 << 24) for v in vals)
    # slot s reads word s & 3 of block s >> 2
    key = (seed & 0xFFFFFFFF, seed >> 32)
    for s in range(24):
        blk = philox.philox4x32_10((s >> 2, 3, step & 0xFFFFFFFF, step >> 32), key)
        assert vals[s] == blk[s & 3] >> 8
    # draft, accept and final slots never collide for K <= 7
    K = 7
    used = [philox.SLOT_DRAFT + j for j in range(K)] + [philox.SLOT_ACCEPT + j for j in range(K)] \
        + [philox.SLOT_FINAL]
    assert len(set(used)) == len(used)


def test_u24_batches_and_uniformity():
    ud = philox.u24_draft(7, 11, 5, 3)
    ua = philox.u24_accept(7, 11, 5, 3)
    assert ud.shape == (5, 3) and ua.shape == (5, 4)
    assert ud[2, 1] == philox.u24(7, 11, 2, philox.SLOT_DRAFT + 1)
    assert ua[4, 3] == philox.u24(7, 11, 4, philox.SLOT_FINAL)
    # crude uniformity: mean of 20000 draws within 5 sigma of 1/2
    u = np.array([philox.u24(1, s, 0, 0) for s in range(20000)]) / 2.0 ** 24
    assert abs(u.mean() - 0.5) < 5 * (1 / np.sqrt(12 * 20000))
