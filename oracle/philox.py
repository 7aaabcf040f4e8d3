"""Philox4x32-10 counter-based generator and the 24-bit uniforms drawn from it.

Philox (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as 1, 2, 3",
SC'11) is a public algorithm.  Ten rounds; each round multiplies two counter words
by fixed odd constants, swaps the halves around and XORs the round key in; the key
is advanced by a Weyl constant between rounds.

How a speculative step addresses the generator (one 128-bit block per group of four
slots):   key     = (seed low 32, seed high 32)
          counter = (slot >> 2, row, step low 32, step high 32)
          word    = block[slot & 3];   u24 = word >> 8;   u = u24 * 2^-24 in [0, 1)
Slots: draft position k (1-based) -> k-1; accept test k -> 8 + (k-1); the final
(residual / bonus) draw -> 16.  Depth K <= 7 keeps the three ranges apart.
"""
from __future__ import annotations

import numpy as np

_M0 = 0xD2511F53
_M1 = 0xCD9E8D57
_W0 = 0x9E3779B9
_W1 = 0xBB67AE85
_MASK = 0xFFFFFFFF

SLOT_DRAFT = 0      # + (k-1)
SLOT_ACCEPT = 8     # + (k-1)
SLOT_FINAL = 16


def philox4x32_10(counter, key):
    """One Philox4x32-10 block.  ``counter``: 4 ints, ``key``: 2 ints (each < 2^32)."""
    c0, c1, c2, c3 = (int(c) & _MASK for c in counter)
    k0, k1 = (int(k) & _MASK for k in key)
    for r in range(10):
        if r > 0:
            k0 = (k0 + _W0) & _MASK
            k1 = (k1 + _W1) & _MASK
        p0 = _M0 * c0
        p1 = _M1 * c2
        hi0, lo0 = p0 >> 32, p0 & _MASK
        hi1, lo1 = p1 >> 32, p1 & _MASK
        c0, c1, c2, c3 = hi1 ^ c1 ^ k0, lo1, hi0 ^ c3 ^ k1, lo0
    return (c0, c1, c2, c3)


def u24(seed: int, step: int, row: int, slot: int) -> int:
    """The 24-bit uniform of (seed, step, row, slot)."""
    key = (seed & _MASK, (seed >> 32) & _MASK)
    ctr = (slot >> 2, row & _MASK, step & _MASK, (step >> 32) & _MASK)
    return philox4x32_10(ctr, key)[slot & 3] >> 8


def u24_draft(seed: int, step: int, batch: int, k: int) -> np.ndarray:
    """Uniforms of the k draft draws of every row: uint32 [batch, k]."""
    return np.array([[u24(seed, step, b, SLOT_DRAFT + j) for j in range(k)]
                     for b in range(batch)], dtype=np.uint32).reshape(batch, k)


def u24_accept(seed: int, step: int, batch: int, k: int) -> np.ndarray:
    """Uniforms of the k accept tests followed by the final draw: uint32 [batch, k+1]."""
    return np.array([[u24(seed, step, b, SLOT_ACCEPT + j) for j in range(k)]
                     + [u24(seed, step, b, SLOT_FINAL)] for b in range(batch)],
                    dtype=np.uint32).reshape(batch, k + 1)
