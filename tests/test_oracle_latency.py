"""Latency expression and hierarchy search against the numbers the paper prints."""
import os

import pytest

from oracle import latency as L

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _load_example(name):
    costs, rows, lat = None, [], []
    for line in open(os.path.join(GOLD, name)):
        p = line.split()
        if not p or p[0].startswith("#"):
            continue
        if p[0] == "costs":
            costs = [float(x) for x in p[1:]]
        elif p[0] == "alpha":
            rows.append([None if x == "-" else float(x) for x in p[1:]])
        elif p[0] == "latency":
            lat.append((int(p[1]), float(p[2]), float(p[3]), p[4] == "pinned"))
    n = len(costs)
    alpha = [[0.0] * n for _ in range(n)]
    for i, r in enumerate(rows):
        for jj, a in enumerate(r):
            if a is not None:
                alpha[i][jj + 1] = a
    return costs, alpha, lat


@pytest.mark.parametrize("name", ["latency_example1.txt", "latency_example2.txt"])
def test_printed_latency_tables(name):
    costs, alpha, lat = _load_example(name)
    n = len(costs)
    checked = 0
    for n_models, printed, tol, pinned in lat:
        idx = list(range(n - n_models, n))
        cc = [costs[i] for i in idx]
        aa = [[alpha[i][j] for j in idx] for i in idx]
        got = L.search_hierarchy(cc, aa, 15)[0]
        if pinned:
            assert abs(got - printed) <= tol, (n_models, got, printed)
            checked += 1
    assert checked >= 2


def test_two_level_closed_forms():
    # Table 1 row 2: target 33, drafter 4, alpha 0.8, best T = 5
    assert abs(L.expected_latency([4, 33], [0.8], [5]) - (1 - 0.8) / (1 - 0.8 ** 6) * (33 + 5 * 4)) < 1e-12
    assert abs(L.expected_latency([4, 33], [0.8], [5]) - 14.37) < 0.005
    assert abs(L.expected_latency([8, 33], [0.8], [3]) - 19.31) < 0.005
    assert L.expected_latency([7.0], [], []) == 7.0


def test_abc_grid():
    lines = [l.split() for l in open(os.path.join(GOLD, "abc_grid.txt")) if l.strip() and not l.startswith("#")]
    costs_c = [float(x) for x in lines[0][1:]]
    cells = off = 0
    for row in lines[1:]:
        a_cb = float(row[0])
        a_ca = max(0.0, a_cb + 0.5 - 1.0)            # triangle-inequality lower bound
        for cost_c, printed in zip(costs_c, row[1:]):
            alpha = [[0, a_cb, a_ca], [0, 0, 0.5], [0, 0, 0]]
            best = L.search_hierarchy([cost_c, 256.0, 1024.0], alpha, 15)[0]
            err = abs(round(1024.0 / best, 2) - float(printed))
            assert err <= 0.0101, (a_cb, cost_c, 1024.0 / best, printed)
            off += err > 0.001
            cells += 1
    assert cells == 80 and off <= 6


def test_gamma_properties():
    assert L.gamma(0.3, 4, 1) == 1.0                       # one round always yields >= 1 token
    assert abs(L.gamma(0.0, 5, 7) - 7.0) < 1e-12           # every draft rejected: 1 token per round
    assert abs(L.gamma(1.0, 2, 6) - 2.0) < 1e-12           # all accepted: 3 tokens per round
    # T_out = 2: one round suffices unless the first draft is rejected
    assert abs(L.gamma(0.6, 3, 2) - (1 + 0.4)) < 1e-12
    # Monte-Carlo check of the renewal reading
    import random
    rnd = random.Random(0)
    tot = 0
    for _ in range(40000):
        have = rounds = 0
        while have < 7:
            k = 1
            while k <= 3 and rnd.random() < 0.7:
                k += 1
            have += min(k, 4)
            rounds += 1
        tot += rounds
    assert abs(tot / 40000 - L.gamma(0.7, 3, 7)) < 0.02


def test_search_equals_brute_force():
    costs = [0.5, 2.0, 6.0, 20.0]
    alpha = [[0, 0.8, 0.6, 0.45], [0, 0, 0.75, 0.6], [0, 0, 0, 0.8], [0] * 4]
    a = L.search_hierarchy(costs, alpha, 5)
    b = L.brute_force_hierarchy(costs, alpha, 5)
    assert abs(a[0] - b[0]) < 1e-12 and a[1] == b[1] and a[2] == b[2]
    # fixed chain, monotone T
    t = L.search_T(costs, [0.8, 0.75, 0.8], 5)
    assert abs(t[0] - L.expected_latency(costs, [0.8, 0.75, 0.8], t[1])) < 1e-15
    assert t[0] >= a[0] - 1e-12
