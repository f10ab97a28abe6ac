"""Pins the oracle's Philox4x32-10 to the published known-answer vectors and
checks the uniform convention of the decode step."""
import os

from oracle import philox

GOLD = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_kat.txt")


def test_known_answer_vectors():
    n = 0
    for line in open(GOLD):
        if line.startswith("#") or not line.strip():
            continue
        w = [int(x, 16) for x in line.split()]
        assert philox.philox4x32_10(w[0:4], w[4:6]) == tuple(w[6:10])
        n += 1
    assert n == 3


def test_uniform_open_interval_and_grid():
    seen = set()
    for pos in range(200):
        u = philox.uniform(1, pos, 0, 0, philox.STREAM_ACCEPT)
        assert 0.0 < u < 1.0
        k = u * 2 ** 24 - 0.5
        assert k == int(k)            # on the 24-bit grid, hence exact in fp32
        seen.add(u)
    assert len(seen) > 190


def test_streams_and_counters_decorrelate():
    a = philox.uniform(1, 5, 0, 0, 0)
    assert a != philox.uniform(1, 5, 0, 0, 1)
    assert a != philox.uniform(1, 5, 1, 0, 0)
    assert a != philox.uniform(1, 5, 0, 1, 0)
    assert a != philox.uniform(2, 5, 0, 0, 0)
    assert a == philox.uniform(1, 5, 0, 0, 0)


def test_uniform_mean_is_half():
    us = [philox.uniform(7, p, 3, s, 0) for p in range(100) for s in range(40)]
    m = sum(us) / len(us)
    assert abs(m - 0.5) < 4 * (1 / 12 / len(us)) ** 0.5
