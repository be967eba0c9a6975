"""Philox4x32-10 against published known-answer vectors."""
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


def test_uniform_addressing_is_order_free_and_distinct():
    # a decision's uniform depends only on its address, and every address field matters
    base = philox.uniform24(5, 1, 2, 1, philox.PURPOSE_ACCEPT, 0)
    assert base == philox.uniform24(5, 1, 2, 1, philox.PURPOSE_ACCEPT, 0)
    others = {philox.uniform24(6, 1, 2, 1, 1, 0), philox.uniform24(5, 2, 2, 1, 1, 0),
              philox.uniform24(5, 1, 3, 1, 1, 0), philox.uniform24(5, 1, 2, 2, 1, 0),
              philox.uniform24(5, 1, 2, 1, 2, 0), philox.uniform24(5, 1, 2, 1, 1, 1),
              philox.uniform24(5 + (1 << 32), 1, 2, 1, 1, 0)}
    assert base not in others and len(others) == 7
    assert 0 <= base < (1 << 24)


def test_uniform_mean_and_spread():
    us = [philox.uniform24(11, j, 0, 0, 0, 0) / 2.0 ** 24 for j in range(20000)]
    m = sum(us) / len(us)
    v = sum((u - m) ** 2 for u in us) / len(us)
    assert abs(m - 0.5) < 0.01 and abs(v - 1.0 / 12.0) < 0.005
