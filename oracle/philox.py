"""Philox4x32-10 counter-based generator, written from the published algorithm
(Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as 1, 2, 3",
SC'11).  TEST INFRASTRUCTURE: part of the CPU oracle; the CUDA library has its
own implementation and shares nothing with this file.

The paper under study does not say how random numbers are drawn for the
accept test (Eq. 2) or the residual draw (Eq. 3); the reading used here is
stated in `uniform01` and `draw_u`.
"""
from __future__ import annotations

MASK32 = 0xFFFFFFFF
PHILOX_M0 = 0xD2511F53
PHILOX_M1 = 0xCD9E8D57
PHILOX_W0 = 0x9E3779B9  # golden ratio
PHILOX_W1 = 0xBB67AE85  # sqrt(3) - 1

# purposes (second counter word)
PURPOSE_DRAFT = 0    # draw of a draft token from q
PURPOSE_ACCEPT = 1   # uniform of the accept test
PURPOSE_EXTRA = 2    # draw of the corrected / bonus / plain autoregressive token


def philox4x32_10(counter, key):
    """counter: 4 uint32, key: 2 uint32 -> 4 uint32 after 10 rounds."""
    c0, c1, c2, c3 = (int(c) & MASK32 for c in counter)
    k0, k1 = (int(k) & MASK32 for k in key)
    for _ in range(10):
        p0 = PHILOX_M0 * c0
        p1 = PHILOX_M1 * c2
        hi0, lo0 = p0 >> 32, p0 & MASK32
        hi1, lo1 = p1 >> 32, p1 & MASK32
        c0, c1, c2, c3 = (hi1 ^ c1 ^ k0) & MASK32, lo1, (hi0 ^ c3 ^ k1) & MASK32, lo0
        k0 = (k0 + PHILOX_W0) & MASK32
        k1 = (k1 + PHILOX_W1) & MASK32
    return c0, c1, c2, c3


def uniform01(x: int) -> float:
    """uint32 -> u in (0,1): the top 23 bits plus one half, times 2^-23.

    u = (2·(x >> 9) + 1) · 2^-24 has an odd 24-bit numerator, so every such
    value is exactly representable in fp32 and a CPU and a GPU implementation
    obtain the same u bit for bit.
    """
    return ((int(x) >> 9) + 0.5) * (1.0 / 8388608.0)


def draw_u(seed: int, seq: int, position: int, purpose: int) -> float:
    """The uniform used for one decision.

    key = the 64-bit seed split in two words; counter = (absolute index of the
    token being decided, purpose, sequence index in the batch, 0).  Keying by
    position makes a draw independent of how rounds happen to be cut.
    """
    key = (seed & MASK32, (seed >> 32) & MASK32)
    out = philox4x32_10((position, purpose, seq, 0), key)
    return uniform01(out[0])
