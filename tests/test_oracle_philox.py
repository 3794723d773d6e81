"""Known-answer test of the oracle's Philox4x32-10 against the vectors published with
the algorithm's reference implementation (tests/golden/philox4x32_10_kat.txt)."""
import os

from oracle import philox


def _vectors():
    path = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_kat.txt")
    for line in open(path):
        if line.startswith("#") or not line.strip():
            continue
        w = [int(x, 16) for x in line.split()]
        yield w[:4], w[4:6], tuple(w[6:])


def test_known_answers():
    n = 0
    for ctr, key, expect in _vectors():
        assert philox.philox4x32_10(ctr, key) == expect
        n += 1
    assert n == 3


def test_draw_u_uses_key_and_counter_words():
    base = philox.draw_u(5, 0, 10, 0)
    assert 0.0 < base < 1.0
    assert base == philox.draw_u(5, 0, 10, 0)
    assert len({base, philox.draw_u(6, 0, 10, 0), philox.draw_u(5, 1, 10, 0),
                philox.draw_u(5, 0, 11, 0), philox.draw_u(5, 0, 10, 1),
                philox.draw_u(5 + (1 << 32), 0, 10, 0)}) == 6
